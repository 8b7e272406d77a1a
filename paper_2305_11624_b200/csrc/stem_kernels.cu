// First-layer ("stem") convolutions: very few input channels (C_in <= 8, e.g. 7x7 stride 2 on RGB).
// A pixel is then only 6-16 bytes, too narrow for TMA and for a 64-wide K block.  The input is first
// repacked to 8 channels per pixel (16 bytes) with an explicit zero border, after which the kw <= 8
// pixels a filter row touches are 128 contiguous bytes: one K row of 64 "channels" (8 pixels x 8
// channels) per filter row r.  A 5-D strided tensor map exposes those overlapping windows to TMA, and
// the dense tensor-core kernels run with K = kh * 64 (zeros in the unused slots of the weights).
#include "kernels.h"

namespace convbn {

bool stem_eligible(const Problem &pb) {
    return pb.groups == 1 && pb.c_in <= 8 && pb.kw <= 8 && pb.kh <= 16 && pb.dil_h == 1 && pb.dil_w == 1 &&
           pb.stride_h <= 4 && pb.stride_w <= 4 && pb.c_out % 64 == 0 && pb.c_out <= 1024 &&
           pb.p < (1LL << 30) && pb.pin < (1LL << 30);
}

void stem_geometry(const Problem &pb, int *hp, int *wp) {
    const int need_h = (pb.h_out - 1) * pb.stride_h + pb.kh, need_w = (pb.w_out - 1) * pb.stride_w + 8;
    const int have_h = pb.h_in + 2 * pb.pad_h, have_w = pb.w_in + 2 * pb.pad_w;
    *hp = need_h > have_h ? need_h : have_h;
    *wp = need_w > have_w ? need_w : have_w;
}

size_t stem_packed_bytes(const Problem &pb) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    return (size_t)pb.n * hp * wp * 16;
}

size_t stem_weight_bytes(const Problem &pb) { return (size_t)pb.c_out * pb.kh * 64 * 2; }

// xp[n][hp][wp][8] = x[n][h - pad_h][w - pad_w][c] inside the image, 0 in the border and for c >= C_in
__global__ void __launch_bounds__(256) stem_pack_kernel(int n, int h_in, int w_in, int c_in, int pad_h, int pad_w,
                                                        int hp, int wp, const __nv_bfloat16 *__restrict__ x,
                                                        uint4 *__restrict__ xp) {
    const long long total = (long long)n * hp * wp;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int wq = (int)(i % wp);
        const long long t = i / wp;
        const int hq = (int)(t % hp), img = (int)(t / hp);
        const int h = hq - pad_h, w = wq - pad_w;
        unsigned short v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (h >= 0 && h < h_in && w >= 0 && w < w_in) {
            const unsigned short *src = (const unsigned short *)x + (((long long)img * h_in + h) * w_in + w) * c_in;
            for (int c = 0; c < c_in; ++c) v[c] = src[c];
        }
        uint4 q;
        q.x = v[0] | ((uint32_t)v[1] << 16); q.y = v[2] | ((uint32_t)v[3] << 16);
        q.z = v[4] | ((uint32_t)v[5] << 16); q.w = v[6] | ((uint32_t)v[7] << 16);
        xp[i] = q;
    }
}

cudaError_t launch_stem_pack(const Problem &pb, const void *x, void *xp, cudaStream_t st) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    const long long total = (long long)pb.n * hp * wp;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    stem_pack_kernel<<<(int)blocks, 256, 0, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.pad_h, pb.pad_w, hp, wp,
                                                  (const __nv_bfloat16 *)x, (uint4 *)xp);
    return cudaGetLastError();
}

// wst[co][r][q * 8 + c] = scale[co] * w[co][r][q][c]  (q < kw, c < C_in), zero elsewhere
__global__ void __launch_bounds__(256) stem_expand_weights_kernel(int c_out, int kh, int kw, int c_in,
                                                                  const __nv_bfloat16 *__restrict__ w,
                                                                  const float *__restrict__ s_vec,
                                                                  __nv_bfloat16 *__restrict__ wst) {
    const int total = c_out * kh * 64;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int j = i & 63, r = (i >> 6) % kh, co = (i >> 6) / kh;
        const int q = j >> 3, c = j & 7;
        float v = 0.f;
        if (q < kw && c < c_in)
            v = (s_vec ? s_vec[co] : 1.f) * __bfloat162float(w[(((long long)co * kh + r) * kw + q) * c_in + c]);
        wst[i] = __float2bfloat16_rn(v);
    }
}

cudaError_t launch_stem_expand_weights(const Problem &pb, const void *w, const float *s_vec, void *wst,
                                       cudaStream_t st) {
    const int total = pb.c_out * pb.kh * 64;
    stem_expand_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(pb.c_out, pb.kh, pb.kw, pb.c_in,
                                                                    (const __nv_bfloat16 *)w, s_vec,
                                                                    (__nv_bfloat16 *)wst);
    return cudaGetLastError();
}

// ---- backward data of a stem layer (plain ALUs) ---------------------------------------------------
// dX[n,h,w,c] = sum over the taps that reach (h, w) and over co of omega'[co,r,q,c] dZ[n,ho,wo,co]
// (Sec. 3.2.1).  With C_in <= 8 the GEMM N dimension is too narrow for the tensor cores, and the first
// layer's input gradient is rarely needed, so this is an fp32 FMA kernel: blockIdx.y is the residue
// class (h mod stride_h, w mod stride_w), so all lanes of a warp meet the same taps and read the
// (scaled, fp32) weights from shared memory as broadcasts; dZ is read 8 channels (16 bytes) at a time.
template <int CP>      // channels kept per thread: C_in rounded up to 4 or 8 (weights zero-padded)
__global__ void __launch_bounds__(256) stem_dgrad_kernel(int n, int h_in, int w_in, int c_in, int h_out, int w_out,
                                                         int c_out, int kh, int kw, int stride_h, int stride_w,
                                                         int pad_h, int pad_w, const uint4 *__restrict__ dz,
                                                         const __nv_bfloat16 *__restrict__ w,
                                                         const float *__restrict__ s_vec,
                                                         __nv_bfloat16 *__restrict__ dx) {
    extern __shared__ float w_s[];                  // [tap][co][CP]
    const int taps = kh * kw;
    for (int i = threadIdx.x; i < taps * c_out * CP; i += blockDim.x) {
        const int c = i % CP, t = i / CP, co = t % c_out, tap = t / c_out;
        w_s[i] = c < c_in ? (s_vec ? s_vec[co] : 1.f) * __bfloat162float(w[((size_t)co * taps + tap) * c_in + c]) : 0.f;
    }
    __syncthreads();
    const int a = blockIdx.y / stride_w, b = blockIdx.y % stride_w;
    if (a >= h_in || b >= w_in) return;
    const int hi_n = (h_in - a + stride_h - 1) / stride_h, wj_n = (w_in - b + stride_w - 1) / stride_w;
    const uint32_t total = (uint32_t)n * hi_n * wj_n;
    const int v = c_out / 8;
    for (uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const uint32_t t1 = idx / (uint32_t)wj_n;
        const int j = (int)(idx - t1 * (uint32_t)wj_n);
        const uint32_t img = t1 / (uint32_t)hi_n;
        const int i = (int)(t1 - img * (uint32_t)hi_n);
        const int h = i * stride_h + a, wq = j * stride_w + b;
        float acc[CP];
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[c] = 0.f;
        for (int r = (a + pad_h) % stride_h; r < kh; r += stride_h) {
            const int hs = h + pad_h - r;
            if (hs < 0) break;
            const int ho = hs / stride_h;
            if (ho >= h_out) continue;
            for (int q = (b + pad_w) % stride_w; q < kw; q += stride_w) {
                const int ws = wq + pad_w - q;
                if (ws < 0) break;
                const int wo = ws / stride_w;
                if (wo >= w_out) continue;
                const uint4 *src = dz + ((size_t)(img * h_out + ho) * w_out + wo) * v;
                const float *wt = w_s + (size_t)(r * kw + q) * c_out * CP;
                for (int g8 = 0; g8 < v; ++g8) {
                    const uint4 qv = __ldg(src + g8);
                    const uint32_t u[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float d = __uint_as_float((e & 1) ? (u[e >> 1] & 0xFFFF0000u) : (u[e >> 1] << 16));
                        const float4 *wc = (const float4 *)(wt + (g8 * 8 + e) * CP);
#pragma unroll
                        for (int c4 = 0; c4 < CP / 4; ++c4) {
                            const float4 wv = wc[c4];
                            acc[4 * c4] = fmaf(d, wv.x, acc[4 * c4]); acc[4 * c4 + 1] = fmaf(d, wv.y, acc[4 * c4 + 1]);
                            acc[4 * c4 + 2] = fmaf(d, wv.z, acc[4 * c4 + 2]); acc[4 * c4 + 3] = fmaf(d, wv.w, acc[4 * c4 + 3]);
                        }
                    }
                }
            }
        }
        __nv_bfloat16 *dst = dx + ((size_t)(img * h_in + h) * w_in + wq) * c_in;
#pragma unroll
        for (int c = 0; c < CP; ++c)
            if (c < c_in) dst[c] = __float2bfloat16_rn(acc[c]);
    }
}

bool stem_dgrad_eligible(const Problem &pb) {
    return stem_eligible(pb) && pb.c_out % 8 == 0 &&
           (size_t)pb.kh * pb.kw * pb.c_out * (pb.c_in <= 4 ? 4 : 8) * sizeof(float) <= 160 * 1024;
}

cudaError_t launch_stem_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                              cudaStream_t st) {
    const int cp = pb.c_in <= 4 ? 4 : 8;
    const size_t smem = (size_t)pb.kh * pb.kw * pb.c_out * cp * sizeof(float);
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(stem_dgrad_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(stem_dgrad_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const long long per_class = (long long)pb.n * ((pb.h_in + pb.stride_h - 1) / pb.stride_h) *
                                ((pb.w_in + pb.stride_w - 1) / pb.stride_w);
    long long bx = (per_class + 255) / 256;
    if (bx > 148 * 8) bx = 148 * 8;
    dim3 grid((unsigned)bx, (unsigned)(pb.stride_h * pb.stride_w));
    if (cp == 4)
        stem_dgrad_kernel<4><<<grid, 256, smem, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.c_out,
                                                      pb.kh, pb.kw, pb.stride_h, pb.stride_w, pb.pad_h, pb.pad_w,
                                                      (const uint4 *)dz, (const __nv_bfloat16 *)w, s_vec,
                                                      (__nv_bfloat16 *)dx);
    else
        stem_dgrad_kernel<8><<<grid, 256, smem, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.c_out,
                                                      pb.kh, pb.kw, pb.stride_h, pb.stride_w, pb.pad_h, pb.pad_w,
                                                      (const uint4 *)dz, (const __nv_bfloat16 *)w, s_vec,
                                                      (__nv_bfloat16 *)dx);
    return cudaGetLastError();
}

}  // namespace convbn
