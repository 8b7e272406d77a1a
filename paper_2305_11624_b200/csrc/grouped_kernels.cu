// Grouped convolution helpers for the block-diagonal tensor-core path (bf16 NHWC, C_in/G = C_out/G = cg,
// cg divides 64, C a multiple of 64).  A grouped convolution with cg = 8 has about 36 FLOP per byte:
// more than the fp32 ALUs can stream at HBM speed, so each 64-channel block is run as a dense 64 -> 64
// GEMM on the tensor cores with zeros outside the cg x cg diagonal blocks.  These kernels build the
// expanded weight operands and finish the parameter gradients from the block-diagonal partials.
#include "kernels.h"

namespace convbn {

// forward operand : wbd[co][tap][j]            = s[co] w[co][tap][j - start(co)]   for j in co's group
// backward operand: wbd[ci][taps-1-tap][j]     = s[co] w[co][tap][ci % cg], co = 64 (ci / 64) + j, same group
// (zeros elsewhere); start(c) = ((c % 64) / cg) cg.
__global__ void __launch_bounds__(256) expand_blockdiag_kernel(int c, int taps, int cg,
                                                               const __nv_bfloat16 *__restrict__ w,
                                                               const float *__restrict__ s_vec,
                                                               __nv_bfloat16 *__restrict__ wbd, int transpose_flip, int f16) {
    const long long total = (long long)c * taps * 64;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(i & 63);
        const long long t = i >> 6;
        const int tap_o = (int)(t % taps), row = (int)(t / taps);
        float val = 0.f;
        if (!transpose_flip) {
            const int co = row, start = ((co & 63) / cg) * cg;
            if (j >= start && j < start + cg)
                val = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((long long)co * taps + tap_o) * cg + (j - start), f16);
        } else {
            const int ci = row, co = (ci & ~63) + j, tap = taps - 1 - tap_o;
            if ((j / cg) == ((ci & 63) / cg))
                val = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((long long)co * taps + tap) * cg + (ci % cg), f16);
        }
        reinterpret_cast<uint16_t *>(wbd)[i] = pack1_h16(val, f16);
    }
}

cudaError_t launch_expand_blockdiag(const Problem &pb, const void *w, const float *s_vec, void *wbd,
                                    bool transpose_flip, cudaStream_t st) {
    const long long total = (long long)pb.c_out * pb.kh * pb.kw * 64;
    long long blocks = (total + 255) / 256;
    if (blocks > device_sm_count() * 8) blocks = device_sm_count() * 8;
    expand_blockdiag_kernel<<<(int)blocks, 256, 0, st>>>(pb.c_out, pb.kh * pb.kw, pb.cg, (const __nv_bfloat16 *)w,
                                                         s_vec, (__nv_bfloat16 *)wbd, transpose_flip ? 1 : 0, call_f16());
    return cudaGetLastError();
}

// One block per output channel, as the dense epilogue: picks the channel's cg x taps entries out of its
// 64-channel block's partial tiles, adds the slices in order, then forms domega, db, dgamma, dbeta
// (Table 2, Tune row) or the plain sums (vec3 == NULL).
__global__ void __launch_bounds__(256) wgrad_epilogue_bd_kernel(int c_out, int taps, int cg,
                                                               const float *__restrict__ part, int splits,
                                                               const float *__restrict__ bsum_part, int bsplits,
                                                               const __nv_bfloat16 *__restrict__ w,
                                                               const float *__restrict__ vec3,
                                                               const float *__restrict__ b,
                                                               const float *__restrict__ mean,
                                                               float *__restrict__ dw, float *__restrict__ db,
                                                               float *__restrict__ dgamma,
                                                               float *__restrict__ dbeta, int f16) {
    __shared__ float red[256];
    const int co = blockIdx.x, kdim = taps * cg, nblk = c_out / 64;
    const int blk = co >> 6, col = co & 63, start = (col / cg) * cg;
    const size_t tile = (size_t)taps * 64 * 64;
    const float s = vec3 ? vec3[co] : 1.f;
    float dot = 0.f;
    for (int k = threadIdx.x; k < kdim; k += blockDim.x) {
        const int tap = k / cg, cig = k - tap * cg;
        const size_t o = ((size_t)tap * 64 + start + cig) * 64 + col;
        float acc = 0.f;
        for (int sp = 0; sp < splits; ++sp) acc += part[((size_t)sp * nblk + blk) * tile + o];
        dw[(size_t)co * kdim + k] = s * acc;
        if (vec3) dot = fmaf(acc, load_h16(w + (size_t)co * kdim + k, f16), dot);
    }
    float bs = 0.f;
    if (bsum_part)
        for (int sp = threadIdx.x; sp < bsplits; sp += blockDim.x) bs += bsum_part[(size_t)sp * c_out + co];
    red[threadIdx.x] = dot;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    const float dot_all = red[0];
    __syncthreads();
    red[threadIdx.x] = bs;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    if (threadIdx.x == 0) {
        const float dsum = red[0];
        if (vec3) {
            const float r = vec3[2 * c_out + co];
            dbeta[co] = dsum;
            if (db) db[co] = s * dsum;
            dgamma[co] = r * (dot_all + dsum * ((b ? b[co] : 0.f) - mean[co]));
        } else if (db) {
            db[co] = dsum;
        }
    }
}

cudaError_t launch_wgrad_epilogue_bd(const Problem &pb, const float *partials, int splits,
                                     const float *bsum_part, int bsplits, const void *w, const float *vec3,
                                     const float *b, const float *mean, float *dw, float *db, float *dgamma,
                                     float *dbeta, cudaStream_t st) {
    wgrad_epilogue_bd_kernel<<<pb.c_out, 256, 0, st>>>(pb.c_out, pb.kh * pb.kw, pb.cg, partials, splits, bsum_part,
                                                       bsplits, (const __nv_bfloat16 *)w, vec3, b, mean, dw, db,
                                                       dgamma, dbeta, call_f16());
    return cudaGetLastError();
}

}  // namespace convbn
