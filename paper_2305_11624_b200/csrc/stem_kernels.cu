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
// layer's input gradient is rarely needed, so this is an fp32 FMA kernel.  A block works on one
// residue class (h mod stride_h, w mod stride_w) at a time, so every lane meets the same taps.  Eight
// lanes share a group of PX pixels of one row: lane l of the eight takes the 8-channel chunks l, l+8,
// ... of dZ, so that a warp's 16-byte loads cover contiguous 128-byte pixels, and the eight partial
// sums meet in a butterfly.  The (scaled, fp32) weights sit in shared memory as
// [tap][chunk/8][channel in chunk][chunk%8][CP], which puts the eight lanes' 16-byte reads side by side;
// each weight read serves PX pixels, and the PX + 3 columns of dZ that four taps of a kernel row need
// are loaded and widened to fp32 once for all four.
template <int CP, int CIN, int PX>   // CP: floats per weight vector (4 or 8); CIN: channels accumulated (<= CP)
__global__ void __launch_bounds__(256) stem_dgrad_kernel(int n, int h_in, int w_in, int c_in, int h_out, int w_out,
                                                         int c_out, int kh, int kw, int stride_h, int stride_w,
                                                         int pad_h, int pad_w, const uint4 *__restrict__ dz,
                                                         const __nv_bfloat16 *__restrict__ w,
                                                         const float *__restrict__ s_vec,
                                                         __nv_bfloat16 *__restrict__ dx) {
    extern __shared__ float w_s[];
    const int taps = kh * kw;
    const int v = c_out / 8, vo = (v + 7) / 8;
#pragma unroll 8
    for (int i = threadIdx.x; i < taps * vo * 64 * CP; i += blockDim.x) {
        const int c = i % CP;
        int t = i / CP;
        const int l = t % 8;
        t /= 8;
        const int e = t % 8;
        t /= 8;
        const int go = t % vo, tap = t / vo;
        const int co = (go * 8 + l) * 8 + e;
        w_s[i] = (co < c_out && c < c_in)
                     ? (s_vec ? s_vec[co] : 1.f) * __bfloat162float(w[((size_t)co * taps + tap) * c_in + c])
                     : 0.f;
    }
    __syncthreads();
    const int l8 = threadIdx.x & 7;
    const uint32_t gpb = blockDim.x >> 3;                      // pixel groups per block and pass
    const size_t tap_floats = (size_t)vo * 64 * CP;
    // Work items are (pass of gpb pixel groups, residue class).  A block owns a contiguous run of
    // passes and visits every class of a pass before the next pass: the classes of one pass, and
    // neighbouring passes, read the same rows of dZ, and every block meets the classes equally often
    // although they have different tap counts.
    const int wq_max = ((w_in + stride_w - 1) / stride_w + PX - 1) / PX;
    const uint32_t ipc = ((uint32_t)n * ((h_in + stride_h - 1) / stride_h) * wq_max + gpb - 1) / gpb;
    const uint32_t ncls = (uint32_t)(stride_h * stride_w);
    const uint32_t run = (ipc + gridDim.x - 1) / gridDim.x;
    const uint32_t pass_end = min(ipc, (blockIdx.x + 1) * run);
    for (uint32_t item = blockIdx.x * run * ncls; item < pass_end * ncls; ++item) {
        const int cls = (int)(item % ncls);
        const uint32_t base = (item / ncls) * gpb;
        const int a = cls / stride_w, b = cls % stride_w;
        if (a >= h_in || b >= w_in) continue;
        const int hi_n = (h_in - a + stride_h - 1) / stride_h, wj_n = (w_in - b + stride_w - 1) / stride_w;
        const int wq_n = (wj_n + PX - 1) / PX;                 // groups of PX pixels along a row
        const uint32_t total = (uint32_t)n * hi_n * wq_n;
        if (base >= total) continue;
        const int r0 = (a + pad_h) % stride_h, q0 = (b + pad_w) % stride_w;
        uint32_t idx = base + (threadIdx.x >> 3);
        const bool live = idx < total;
        if (!live) idx = total - 1;                            // keeps the whole warp in the butterfly
        const uint32_t t1 = idx / (uint32_t)wq_n;
        const int j = (int)(idx - t1 * (uint32_t)wq_n) * PX;
        const uint32_t img = t1 / (uint32_t)hi_n;
        const int i = (int)(t1 - img * (uint32_t)hi_n);
        const int h = i * stride_h + a, wq = j * stride_w + b;
        float acc[PX][CIN];
#pragma unroll
        for (int p = 0; p < PX; ++p)
#pragma unroll
            for (int c = 0; c < CIN; ++c) acc[p][c] = 0.f;
        for (int g8 = l8; g8 < v; g8 += 8) {
            const float *wg = w_s + ((size_t)(g8 >> 3) * 64 + l8) * CP;
            for (int r = r0; r < kh; r += stride_h) {
                // h + pad_h - r and wq + pad_w - q are multiples of the stride inside a class, also when negative
                const int ho = (h + pad_h - r) / stride_h;
                if (ho < 0 || ho >= h_out) continue;
                const uint4 *row = dz + ((size_t)(img * h_out + ho) * w_out) * v + g8;
                for (int qb = q0; qb < kw; qb += 4 * stride_w) {
                    // Four taps of one kernel row at a time: tap u of them pairs pixel p with output column
                    // wo0 - u + p, so the PX + 3 columns from wo0 - 3 on serve all four taps.
                    const int wo0 = (wq + pad_w - qb) / stride_w;
                    const int nu = min(4, (kw - qb + stride_w - 1) / stride_w);
                    uint4 win[PX + 3];
#pragma unroll
                    for (int k = 0; k < PX + 3; ++k) {
                        const int wk = wo0 - 3 + k;
                        win[k] = (k >= 4 - nu && wk >= 0 && wk < w_out) ? __ldg(row + (size_t)wk * v)
                                                                         : make_uint4(0u, 0u, 0u, 0u);
                    }
                    const float *wt = wg + (size_t)(r * kw + qb) * tap_floats;
                    const size_t tap_step = (size_t)stride_w * tap_floats;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {              // channel e of the lane's chunk, widened once
                        float d[PX + 3];
#pragma unroll
                        for (int k = 0; k < PX + 3; ++k) {
                            const uint32_t word = e < 2 ? win[k].x : e < 4 ? win[k].y : e < 6 ? win[k].z : win[k].w;
                            d[k] = __uint_as_float((e & 1) ? (word & 0xFFFF0000u) : (word << 16));
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (u < nu) {                      // the same for every lane
                                const float4 *wc = (const float4 *)(wt + u * tap_step + e * 8 * CP);
                                float wv[CP];
#pragma unroll
                                for (int c4 = 0; c4 < CP / 4; ++c4) {
                                    const float4 f = wc[c4];
                                    wv[4 * c4] = f.x; wv[4 * c4 + 1] = f.y; wv[4 * c4 + 2] = f.z; wv[4 * c4 + 3] = f.w;
                                }
#pragma unroll
                                for (int p = 0; p < PX; ++p)
#pragma unroll
                                    for (int c = 0; c < CIN; ++c) acc[p][c] = fmaf(d[p - u + 3], wv[c], acc[p][c]);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int p = 0; p < PX; ++p) {
            float mine = 0.f;
#pragma unroll
            for (int c = 0; c < CIN; ++c) {
                float t = acc[p][c];
                t += __shfl_xor_sync(0xFFFFFFFFu, t, 1);
                t += __shfl_xor_sync(0xFFFFFFFFu, t, 2);
                t += __shfl_xor_sync(0xFFFFFFFFu, t, 4);
                if (l8 == c) mine = t;
            }
            if (live && j + p < wj_n && l8 < c_in)
                dx[((size_t)(img * h_in + h) * w_in + wq + p * stride_w) * c_in + l8] = __float2bfloat16_rn(mine);
        }
    }
}

bool stem_dgrad_eligible(const Problem &pb) {
    return stem_eligible(pb) && pb.c_out % 8 == 0 &&
           (size_t)pb.kh * pb.kw * ((pb.c_out / 8 + 7) / 8) * 64 * (pb.c_in <= 4 ? 4 : 8) * sizeof(float) <= 160 * 1024;
}

cudaError_t launch_stem_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                              cudaStream_t st) {
    const int cp = pb.c_in <= 4 ? 4 : 8;
    const int vo = (pb.c_out / 8 + 7) / 8;
    const size_t smem = (size_t)pb.kh * pb.kw * vo * 64 * cp * sizeof(float);
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(stem_dgrad_kernel<4, 3, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(stem_dgrad_kernel<4, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(stem_dgrad_kernel<8, 8, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const long long passes = ((long long)pb.n * pb.h_in * pb.w_in + 63) / 64;
    const unsigned grid = (unsigned)(passes < 148 * 2 ? passes : 148 * 2);   // two resident blocks per SM
#define CONVBN_STEM_DGRAD(CP_, CIN_, PX_)                                                                           \
    stem_dgrad_kernel<CP_, CIN_, PX_><<<grid, 256, smem, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out,     \
                                                          pb.c_out, pb.kh, pb.kw, pb.stride_h, pb.stride_w,        \
                                                          pb.pad_h, pb.pad_w, (const uint4 *)dz,                   \
                                                          (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)dx)
    if (pb.c_in == 3) CONVBN_STEM_DGRAD(4, 3, 8);
    else if (cp == 4) CONVBN_STEM_DGRAD(4, 4, 4);
    else CONVBN_STEM_DGRAD(8, 8, 4);
#undef CONVBN_STEM_DGRAD
    return cudaGetLastError();
}

}  // namespace convbn
