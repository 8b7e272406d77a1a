// Depthwise ConvBN kernels (groups = C_in = C_out), bf16 NHWC, C a multiple of 8.
// Depthwise convolution has about 4.5 FLOP per byte: it is a streaming problem, so these kernels use
// the plain ALUs with 128-bit (8-channel) coalesced accesses along C and keep fp32 accumulators in
// registers; neighbouring taps are served by L1.
//   forward        Z[n,h,w,c]  = b'[c] + sum_{r,q} omega'[c,r,q] X[n, h s - p + r d, w s - p + q d, c]   (Sec. 3.1/3.3)
//   backward data  dX = omega'_rot (*) dZ   (Sec. 3.2.1), gathered per dX element
//   backward weight domega'[c,r,q] = sum_{n,h,w} dZ[n,h,w,c] X[n, ...]   (Sec. 3.2.1), per-slice partials
#include <cstdlib>

#include "kernels.h"
#include "packed_f32.cuh"

namespace convbn {

namespace {

constexpr int kMaxTaps = 49;   // up to 7 x 7

struct DwShape {
    int n, c, h_in, w_in, h_out, w_out, kh, kw, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
    int f16;               // 16-bit storage type: 0 bf16, 1 IEEE half
};

__device__ __forceinline__ void unpack8(const uint4 &q, float (&f)[8], int f16) {
    const uint32_t u[4] = {q.x, q.y, q.z, q.w};
    if (f16) {
#pragma unroll
        for (int e = 0; e < 4; ++e) unpack2_t<true>(u[e], f[2 * e], f[2 * e + 1]);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) unpack2_t<false>(u[e], f[2 * e], f[2 * e + 1]);
    }
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8], int f16) {
    return make_uint4(pack2_h16(f[0], f[1], f16), pack2_h16(f[2], f[3], f16), pack2_h16(f[4], f[5], f16),
                      pack2_h16(f[6], f[7], f16));
}

// Stage the block's weights in shared memory as fp32 [tap][C] (global layout is [C][tap]).
__device__ __forceinline__ void stage_weights(float *w_s, const __nv_bfloat16 *w, int taps, int c, int f16) {
    for (int i = threadIdx.x; i < taps * c; i += blockDim.x) {
        const int ch = i % c, t = i / c;
        w_s[i] = load_h16(w + (size_t)ch * taps + t, f16);
    }
    __syncthreads();
}

// One thread: 8 channels x TW consecutive output columns of one output row.  For unit stride and
// dilation along W the TW + kw - 1 input vectors of a row are loaded once and reused by all taps.
template <int TW, int KW>
__global__ void __launch_bounds__(256) dw_fwd_kernel(DwShape s, const uint4 *__restrict__ x,
                                                     const __nv_bfloat16 *__restrict__ w,
                                                     const float *__restrict__ bias, uint4 *__restrict__ z) {
    extern __shared__ float w_s[];                   // [taps][C]
    const int v = s.c / 8;
    stage_weights(w_s, w, s.kh * s.kw, s.c, s.f16);
    const uint32_t wgroups = (uint32_t)(s.w_out + TW - 1) / TW;
    const uint32_t total = (uint32_t)s.n * s.h_out * wgroups * v;
    for (uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        uint32_t t = idx / (uint32_t)v;
        const int cv = (int)(idx - t * (uint32_t)v);
        const uint32_t t1 = t / wgroups;
        const int wg = (int)(t - t1 * wgroups);
        const uint32_t n = t1 / (uint32_t)s.h_out;
        const int ho = (int)(t1 - n * (uint32_t)s.h_out);
        const int wo0 = wg * TW;
        float acc[TW][8];
#pragma unroll
        for (int j = 0; j < TW; ++j)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[j][e] = bias ? bias[cv * 8 + e] : 0.f;
        for (int r = 0; r < s.kh; ++r) {
            const int hi = ho * s.stride_h - s.pad_h + r * s.dil_h;
            if (hi < 0 || hi >= s.h_in) continue;
            const uint4 *xrow = x + ((size_t)(n * s.h_in + hi) * s.w_in) * v + cv;
            if (KW > 0) {
                // unit stride / dilation along W, kw == KW: sliding window in registers
                uint4 seg[TW + (KW > 0 ? KW : 1) - 1];
                const int wi0 = wo0 - s.pad_w;
#pragma unroll
                for (int j = 0; j < TW + KW - 1; ++j) {
                    const int wi = wi0 + j;
                    seg[j] = (wi >= 0 && wi < s.w_in) ? __ldg(xrow + (size_t)wi * v) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int q = 0; q < KW; ++q) {
                    float wv[8];
                    const float *wp = w_s + (r * KW + q) * s.c + cv * 8;
#pragma unroll
                    for (int e = 0; e < 8; ++e) wv[e] = wp[e];
#pragma unroll
                    for (int j = 0; j < TW; ++j) {
                        float xv[8];
                        unpack8(seg[j + q], xv, s.f16);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[j][e] = fmaf(xv[e], wv[e], acc[j][e]);
                    }
                }
            } else {
                for (int q = 0; q < s.kw; ++q) {
                    float wv[8];
                    const float *wp = w_s + (r * s.kw + q) * s.c + cv * 8;
#pragma unroll
                    for (int e = 0; e < 8; ++e) wv[e] = wp[e];
#pragma unroll
                    for (int j = 0; j < TW; ++j) {
                        const int wi = (wo0 + j) * s.stride_w - s.pad_w + q * s.dil_w;
                        if (wi >= 0 && wi < s.w_in && wo0 + j < s.w_out) {
                            float xv[8];
                            unpack8(__ldg(xrow + (size_t)wi * v), xv, s.f16);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[j][e] = fmaf(xv[e], wv[e], acc[j][e]);
                        }
                    }
                }
            }
        }
        uint4 *zrow = z + ((size_t)(n * s.h_out + ho) * s.w_out + wo0) * v + cv;
#pragma unroll
        for (int j = 0; j < TW; ++j)
            if (wo0 + j < s.w_out) zrow[(size_t)j * v] = pack8(acc[j], s.f16);
    }
}

// Unit stride and dilation, KH x KW known at compile time.  One thread: 8 channels x TW output columns,
// walking down `th` output rows.  Every input row of the band is loaded and widened to fp32 once and
// feeds the KH output rows it reaches, whose accumulators rotate through KH register slots; an output
// row is stored when its last input row has been added.
template <int TW, int KH, int KW>
__global__ void __launch_bounds__(256, KH <= 3 ? 2 : 1) dw_stream_kernel(DwShape s, const uint4 *__restrict__ x,
                                                        const __nv_bfloat16 *__restrict__ w,
                                                        const float *__restrict__ bias, uint4 *__restrict__ z,
                                                        int th) {
    extern __shared__ float w_s[];                   // [taps][C]
    constexpr int PF = 3;                            // rows of look-ahead for the L2 prefetch
    const int v = s.c / 8;
    stage_weights(w_s, w, KH * KW, s.c, s.f16);
    const uint32_t wgroups = (uint32_t)(s.w_out + TW - 1) / TW, bands = (uint32_t)(s.h_out + th - 1) / th;
    const uint32_t total = (uint32_t)s.n * bands * wgroups * v;
    for (uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        uint32_t t = idx / (uint32_t)v;
        const int cv = (int)(idx - t * (uint32_t)v);
        const uint32_t t1 = t / wgroups;
        const int wo0 = (int)(t - t1 * wgroups) * TW;
        const uint32_t n = t1 / bands;
        const int ho0 = (int)(t1 - n * bands) * th;
        const int rows = min(th, s.h_out - ho0);
        float bv[8];
        if (bias) {
            const float4 b0 = *reinterpret_cast<const float4 *>(bias + cv * 8);
            const float4 b1 = *reinterpret_cast<const float4 *>(bias + cv * 8 + 4);
            bv[0] = b0.x; bv[1] = b0.y; bv[2] = b0.z; bv[3] = b0.w; bv[4] = b1.x; bv[5] = b1.y; bv[6] = b1.z; bv[7] = b1.w;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) bv[e] = 0.f;
        }
        float acc[KH][TW][8];
#pragma unroll
        for (int sl = 0; sl < KH; ++sl)
#pragma unroll
            for (int j = 0; j < TW; ++j)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[sl][j][e] = bv[e];
        const float *wch = w_s + cv * 8;
        const int wi0 = wo0 - s.pad_w;
        const uint4 *xcol = x + ((size_t)n * s.h_in * s.w_in) * v + cv;
        uint4 *zcol = z + ((size_t)(n * s.h_out + ho0) * s.w_out + wo0) * v + cv;
        // step k brings input row ho0 - pad_h + k, which is tap row r of output row ho0 + k - r;
        // output row o of the band lives in slot o % KH, and k0 is a multiple of KH
        for (int k0 = 0; k0 < rows + KH - 1; k0 += KH) {
#pragma unroll
            for (int ph = 0; ph < KH; ++ph) {
                const int k = k0 + ph;
                if (k < rows + KH - 1) {
                    const int hi = ho0 - s.pad_h + k;
                    if (k + PF < rows + KH - 1 && hi + PF >= 0 && hi + PF < s.h_in) {
                        // ask L2 for the row needed PF steps from now: the loads below then find it there
                        const uint4 *prow = xcol + (size_t)(hi + PF) * s.w_in * v;
#pragma unroll
                        for (int j = 0; j < TW + KW - 1; ++j) {
                            const int wi = wi0 + j;
                            if (wi >= 0 && wi < s.w_in) asm volatile("prefetch.global.L2 [%0];" ::"l"(prow + (size_t)wi * v));
                        }
                    }
                    if (hi >= 0 && hi < s.h_in) {
                        const uint4 *xrow = xcol + (size_t)hi * s.w_in * v;
                        float xs[TW + KW - 1][8];
#pragma unroll
                        for (int j = 0; j < TW + KW - 1; ++j) {
                            const int wi = wi0 + j;
                            unpack8((wi >= 0 && wi < s.w_in) ? __ldg(xrow + (size_t)wi * v) : make_uint4(0, 0, 0, 0), xs[j], s.f16);
                        }
#pragma unroll
                        for (int r = 0; r < KH; ++r) {
                            const int o = k - r;
                            if (o >= 0 && o < rows) {
                                const int sl = (ph - r + KH) % KH;
#pragma unroll
                                for (int q = 0; q < KW; ++q) {
                                    const float4 w0 = *reinterpret_cast<const float4 *>(wch + (r * KW + q) * s.c);
                                    const float4 w1 = *reinterpret_cast<const float4 *>(wch + (r * KW + q) * s.c + 4);
                                    const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                                    for (int j = 0; j < TW; ++j)
#pragma unroll
                                        for (int e = 0; e < 8; ++e) acc[sl][j][e] = fmaf(xs[j + q][e], wv[e], acc[sl][j][e]);
                                }
                            }
                        }
                    }
                    const int od = k - (KH - 1);               // the output row that is complete now
                    if (od >= 0) {
                        const int sl = (ph + 1) % KH;
#pragma unroll
                        for (int j = 0; j < TW; ++j) {
                            if (wo0 + j < s.w_out) zcol[((size_t)od * s.w_out + j) * v] = pack8(acc[sl][j], s.f16);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[sl][j][e] = bv[e];
                        }
                    }
                }
            }
        }
    }
}

// Unit stride and dilation, small KH x KW known at compile time.  One thread: 4 channels x TW output
// columns, walking down `th` output rows, with its KH x KW x 4 weights in registers.  Every input row
// of the band is loaded once, KH rows ahead of its use, into a ring of KH register rows, widened to
// fp32 once and added into the KH output rows it reaches, whose accumulators rotate through KH register
// slots; an output row starts from the bias in its first FMA and is stored when its last input row has
// been added.  Both rings are indexed statically (the row loop is unrolled KH times).  The arithmetic
// is packed fp32 (two channels per FMA instruction).  EDGE: the thread's columns touch the left or right
// border and need per-column guards.
template <int TW, int KH, int KW, bool EDGE>
__device__ __forceinline__ void dw_stream4_item(const DwShape &s, const uint2 *__restrict__ xp, ptrdiff_t pitch,
                                                ptrdiff_t colstep, uint2 *__restrict__ zp, ptrdiff_t zpitch,
                                                int hi0, int rows, int wi0, int wo0, const f32x2 (&wr)[KH * KW][2],
                                                const f32x2 (&bv)[2]) {
    constexpr int NX = TW + KW - 1;
    const uint2 zero = make_uint2(0u, 0u);
    bool col_ok[NX];
#pragma unroll
    for (int j = 0; j < NX; ++j) col_ok[j] = !EDGE || (wi0 + j >= 0 && wi0 + j < s.w_in);
    bool out_ok[TW];
#pragma unroll
    for (int j = 0; j < TW; ++j) out_ok[j] = !EDGE || wo0 + j < s.w_out;
    const int steps = rows + KH - 1;                           // input rows of the band
    uint2 raw[KH][NX];
    f32x2 acc[KH][TW][2];
#pragma unroll
    for (int sl = 0; sl < KH; ++sl) {
        const int hi = hi0 + sl;
        const bool ok = sl < steps && hi >= 0 && hi < s.h_in;
#pragma unroll
        for (int j = 0; j < NX; ++j) raw[sl][j] = (ok && col_ok[j]) ? __ldg(xp + hi * pitch + j * colstep) : zero;
#pragma unroll
        for (int j = 0; j < TW; ++j) acc[sl][j][0] = acc[sl][j][1] = 0ull;
    }
    // step k brings input row hi0 + k, which is tap row r of output row k - r of the band; output row o
    // lives in slot o % KH, input row k in ring row k % KH, and k0 is a multiple of KH
    for (int k0 = 0; k0 < steps; k0 += KH) {
#pragma unroll
        for (int ph = 0; ph < KH; ++ph) {
            const int k = k0 + ph;
            if (k < steps) {
                f32x2 xs[NX][2];
#pragma unroll
                for (int j = 0; j < NX; ++j) xs[j][0] = widen_h16(raw[ph][j].x, s.f16), xs[j][1] = widen_h16(raw[ph][j].y, s.f16);
                {
                    const int hi = hi0 + k + KH;
                    if (k + KH < steps && hi >= 0 && hi < s.h_in) {
#pragma unroll
                        for (int j = 0; j < NX; ++j)
                            raw[ph][j] = col_ok[j] ? __ldg(xp + hi * pitch + j * colstep) : zero;
                    } else {
#pragma unroll
                        for (int j = 0; j < NX; ++j) raw[ph][j] = zero;
                    }
                }
                // tap row 0 opens output row k in slot ph (from the bias); rows before the band's first
                // or past its last only reach slots that are re-opened before, or never reach, a store
#pragma unroll
                for (int r = 0; r < KH; ++r) {
                    const int sl = (ph - r + KH) % KH;
#pragma unroll
                    for (int q = 0; q < KW; ++q)
#pragma unroll
                        for (int j = 0; j < TW; ++j) {
                            acc[sl][j][0] = fma2(xs[j + q][0], wr[r * KW + q][0], (r == 0 && q == 0) ? bv[0] : acc[sl][j][0]);
                            acc[sl][j][1] = fma2(xs[j + q][1], wr[r * KW + q][1], (r == 0 && q == 0) ? bv[1] : acc[sl][j][1]);
                        }
                }
                if (k >= KH - 1) {                             // output row k - (KH - 1) is complete
                    const int sl = (ph + 1) % KH;
                    uint2 *zr = zp + (k - (KH - 1)) * zpitch;
#pragma unroll
                    for (int j = 0; j < TW; ++j)
                        if (out_ok[j]) zr[j * colstep] = make_uint2(narrow_h16(acc[sl][j][0], s.f16), narrow_h16(acc[sl][j][1], s.f16));
                }
            }
        }
    }
}

template <int TW, int KH, int KW>
__global__ void __launch_bounds__(256, 2) dw_stream4_kernel(DwShape s, const uint2 *__restrict__ x,
                                                            const __nv_bfloat16 *__restrict__ w,
                                                            const float *__restrict__ bias, uint2 *__restrict__ z,
                                                            int th) {
    extern __shared__ float w_s[];                   // [taps][C]
    const int v = s.c / 4;
    stage_weights(w_s, w, KH * KW, s.c, s.f16);
    const uint32_t wgroups = (uint32_t)(s.w_out + TW - 1) / TW, bands = (uint32_t)(s.h_out + th - 1) / th;
    const uint32_t total = (uint32_t)s.n * bands * wgroups * v;
    for (uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        uint32_t t = idx / (uint32_t)v;
        const int cv = (int)(idx - t * (uint32_t)v);
        const uint32_t t1 = t / wgroups;
        const int wo0 = (int)(t - t1 * wgroups) * TW;
        const uint32_t n = t1 / bands;
        const int ho0 = (int)(t1 - n * bands) * th;
        const int rows = min(th, s.h_out - ho0);
        f32x2 wr[KH * KW][2];
#pragma unroll
        for (int tp = 0; tp < KH * KW; ++tp) {
            const float4 f = *reinterpret_cast<const float4 *>(w_s + tp * s.c + cv * 4);
            wr[tp][0] = pair(f.x, f.y);
            wr[tp][1] = pair(f.z, f.w);
        }
        f32x2 bv[2] = {0ull, 0ull};
        if (bias) {
            const float4 f = *reinterpret_cast<const float4 *>(bias + cv * 4);
            bv[0] = pair(f.x, f.y);
            bv[1] = pair(f.z, f.w);
        }
        const int wi0 = wo0 - s.pad_w;
        // pointer to (image n, row 0, column wi0): may lie outside the row, and is only dereferenced
        // at columns and rows that are inside
        const uint2 *xp = x + ((ptrdiff_t)n * s.h_in * s.w_in + wi0) * v + cv;
        uint2 *zp = z + ((size_t)(n * s.h_out + ho0) * s.w_out + wo0) * v + cv;
        const bool edge = wi0 < 0 || wi0 + TW + KW - 1 > s.w_in || wo0 + TW > s.w_out;
        if (edge)
            dw_stream4_item<TW, KH, KW, true>(s, xp, (ptrdiff_t)s.w_in * v, v, zp, (ptrdiff_t)s.w_out * v, ho0 - s.pad_h,
                                              rows, wi0, wo0, wr, bv);
        else
            dw_stream4_item<TW, KH, KW, false>(s, xp, (ptrdiff_t)s.w_in * v, v, zp, (ptrdiff_t)s.w_out * v,
                                               ho0 - s.pad_h, rows, wi0, wo0, wr, bv);
    }
}

// dX[n,h,w,c] = sum over taps with (h + p - r d) divisible by the stride of omega'[c,r,q] dZ[n,ho,wo,c].
__global__ void __launch_bounds__(256) dw_dgrad_kernel(DwShape s, const uint4 *__restrict__ dz,
                                                       const __nv_bfloat16 *__restrict__ w,
                                                       uint4 *__restrict__ dx) {
    extern __shared__ float w_s[];
    const int v = s.c / 8;
    stage_weights(w_s, w, s.kh * s.kw, s.c, s.f16);
    const uint32_t total = (uint32_t)s.n * s.h_in * s.w_in * v;
    for (uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        uint32_t t = idx / (uint32_t)v;
        const int cv = (int)(idx - t * (uint32_t)v);
        const uint32_t t1 = t / (uint32_t)s.w_in;
        const int wq = (int)(t - t1 * (uint32_t)s.w_in);
        const uint32_t n = t1 / (uint32_t)s.h_in;
        const int h = (int)(t1 - n * (uint32_t)s.h_in);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int r = 0; r < s.kh; ++r) {
            const int hs = h + s.pad_h - r * s.dil_h;
            if (hs < 0 || hs % s.stride_h) continue;
            const int ho = hs / s.stride_h;
            if (ho >= s.h_out) continue;
            for (int q = 0; q < s.kw; ++q) {
                const int ws = wq + s.pad_w - q * s.dil_w;
                if (ws < 0 || ws % s.stride_w) continue;
                const int wo = ws / s.stride_w;
                if (wo >= s.w_out) continue;
                float dv[8];
                unpack8(__ldg(dz + ((size_t)(n * s.h_out + ho) * s.w_out + wo) * v + cv), dv, s.f16);
                const float *wp = w_s + (r * s.kw + q) * s.c + cv * 8;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(dv[e], wp[e], acc[e]);
            }
        }
        dx[idx] = pack8(acc, s.f16);
    }
}

// Per-slice partials of domega': block = (C/8 channel vectors) x (pixel lanes); every thread keeps
// taps x 8 fp32 sums for its channels over the pixels it visits, then the pixel lanes are added in
// lane order through shared memory.  part[split][c][tap].
template <int TAPS>
__global__ void __launch_bounds__(256) dw_wgrad_kernel(DwShape s, const uint4 *__restrict__ dz,
                                                       const uint4 *__restrict__ x, float *__restrict__ part,
                                                       uint32_t pix_per_block) {
    extern __shared__ float red[];                   // [lanes][v][8]
    const int v = s.c / 8, lanes = blockDim.x / v;
    const int cv = threadIdx.x % v, pl = threadIdx.x / v;
    const uint32_t p_total = (uint32_t)s.n * s.h_out * s.w_out;
    const uint32_t p0 = blockIdx.x * pix_per_block;
    const uint32_t p1 = p0 + pix_per_block < p_total ? p0 + pix_per_block : p_total;
    float acc[TAPS][8];
#pragma unroll
    for (int t = 0; t < TAPS; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = 0.f;
    for (uint32_t p = p0 + pl; p < p1; p += lanes) {
        const uint32_t t2 = p / (uint32_t)s.w_out;
        const int wo = (int)(p - t2 * (uint32_t)s.w_out);
        const uint32_t n = t2 / (uint32_t)s.h_out;
        const int ho = (int)(t2 - n * (uint32_t)s.h_out);
        float dv[8];
        unpack8(__ldg(dz + (size_t)p * v + cv), dv, s.f16);
#pragma unroll
        for (int t = 0; t < TAPS; ++t) {
            const int r = t / s.kw, q = t - r * s.kw;
            const int hi = ho * s.stride_h - s.pad_h + r * s.dil_h;
            const int wi = wo * s.stride_w - s.pad_w + q * s.dil_w;
            if (hi >= 0 && hi < s.h_in && wi >= 0 && wi < s.w_in) {
                float xv[8];
                unpack8(__ldg(x + ((size_t)(n * s.h_in + hi) * s.w_in + wi) * v + cv), xv, s.f16);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[t][e] = fmaf(dv[e], xv[e], acc[t][e]);
            }
        }
    }
#pragma unroll
    for (int t = 0; t < TAPS; ++t) {
#pragma unroll
        for (int e = 0; e < 8; ++e) red[((size_t)pl * v + cv) * 8 + e] = acc[t][e];
        __syncthreads();
        for (int i = threadIdx.x; i < s.c; i += blockDim.x) {
            const int g = i / 8, e = i % 8;
            float sum = 0.f;
            for (int l = 0; l < lanes; ++l) sum += red[((size_t)l * v + g) * 8 + e];
            part[((size_t)blockIdx.x * s.c + i) * TAPS + t] = sum;
        }
        __syncthreads();
    }
}

// Unit stride / dilation, KH x KW known at compile time: every thread requests the
// KH x (TW + KW - 1) input window and TW dZ vectors of its item before any arithmetic.
// Items are (image, output row, group of TW output columns); a block owns a contiguous item range.
template <int TW, int KH, int KW>
__global__ void __launch_bounds__(256, 1) dw_wgrad_window_kernel(DwShape s, const uint4 *__restrict__ dz,
                                                                 const uint4 *__restrict__ x,
                                                                 float *__restrict__ part, uint32_t items_per_block) {
    extern __shared__ float red[];                   // [lanes][v][8]
    constexpr int TAPS = KH * KW;
    const int v = s.c / 8, lanes = blockDim.x / v;
    const int cv = threadIdx.x % v, pl = threadIdx.x / v;
    const uint32_t wgroups = (uint32_t)(s.w_out + TW - 1) / TW;
    const uint32_t items = (uint32_t)s.n * s.h_out * wgroups;
    const uint32_t i0 = blockIdx.x * items_per_block;
    const uint32_t i1 = i0 + items_per_block < items ? i0 + items_per_block : items;
    float acc[TAPS][8];
#pragma unroll
    for (int t = 0; t < TAPS; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = 0.f;
    for (uint32_t it = i0 + pl; it < i1; it += lanes) {
        const uint32_t t1 = it / wgroups;
        const int wg = (int)(it - t1 * wgroups);
        const uint32_t n = t1 / (uint32_t)s.h_out;
        const int ho = (int)(t1 - n * (uint32_t)s.h_out);
        const int wo0 = wg * TW, wi0 = wo0 - s.pad_w, hi0 = ho - s.pad_h;
        uint4 dq[TW], seg[KH][TW + KW - 1];
        const uint4 *drow = dz + ((size_t)(n * s.h_out + ho) * s.w_out + wo0) * v + cv;
#pragma unroll
        for (int j = 0; j < TW; ++j) dq[j] = (wo0 + j < s.w_out) ? __ldg(drow + (size_t)j * v) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int r = 0; r < KH; ++r) {
            const int hi = hi0 + r;
            const bool row_ok = hi >= 0 && hi < s.h_in;
            const uint4 *xrow = x + ((size_t)(n * s.h_in + (row_ok ? hi : 0)) * s.w_in) * v + cv;
#pragma unroll
            for (int j = 0; j < TW + KW - 1; ++j) {
                const int wi = wi0 + j;
                seg[r][j] = (row_ok && wi >= 0 && wi < s.w_in) ? __ldg(xrow + (size_t)wi * v) : make_uint4(0, 0, 0, 0);
            }
        }
        float dv[TW][8];
#pragma unroll
        for (int j = 0; j < TW; ++j) unpack8(dq[j], dv[j], s.f16);
#pragma unroll
        for (int r = 0; r < KH; ++r)
#pragma unroll
            for (int j = 0; j < TW + KW - 1; ++j) {
                float xv[8];
                unpack8(seg[r][j], xv, s.f16);
#pragma unroll
                for (int q = 0; q < KW; ++q) {
                    const int o = j - q;
                    if (o >= 0 && o < TW) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[r * KW + q][e] = fmaf(dv[o][e], xv[e], acc[r * KW + q][e]);
                    }
                }
            }
    }
#pragma unroll
    for (int t = 0; t < TAPS; ++t) {
#pragma unroll
        for (int e = 0; e < 8; ++e) red[((size_t)pl * v + cv) * 8 + e] = acc[t][e];
        __syncthreads();
        for (int i = threadIdx.x; i < s.c; i += blockDim.x) {
            const int g = i / 8, e = i % 8;
            float sum = 0.f;
            for (int l = 0; l < lanes; ++l) sum += red[((size_t)l * v + g) * 8 + e];
            part[((size_t)blockIdx.x * s.c + i) * TAPS + t] = sum;
        }
        __syncthreads();
    }
}

DwShape dw_shape(const Problem &pb) {
    return DwShape{pb.n, pb.c_in, pb.h_in, pb.w_in, pb.h_out, pb.w_out, pb.kh, pb.kw, pb.stride_h, pb.stride_w,
                   pb.pad_h, pb.pad_w, pb.dil_h, pb.dil_w, call_f16()};
}

int dw_grid(long long total) {
    long long b = (total + 255) / 256;
    const long long cap = (long long)device_sm_count() * 32;
    return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

template <class K>
cudaError_t set_smem_once(K kernel, PerDevice *done) { return max_dynamic_smem_once(kernel, 96 * 1024, done); }

}  // namespace

bool dw_eligible(const Problem &pb) {
    return pb.groups == pb.c_in && pb.c_in == pb.c_out && pb.c_in % 8 == 0 && pb.c_in / 8 <= 256 &&
           pb.kh * pb.kw <= kMaxTaps && (size_t)pb.kh * pb.kw * pb.c_in * sizeof(float) <= 96 * 1024 &&
           pb.pin * pb.c_in < (1LL << 31) && pb.p * pb.c_out < (1LL << 31);
}

cudaError_t launch_dw_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                          cudaStream_t st) {
    const DwShape s = dw_shape(pb);
    const size_t smem = (size_t)pb.kh * pb.kw * pb.c_in * sizeof(float);
    const long long total = (long long)pb.n * pb.h_out * ((pb.w_out + 3) / 4) * (pb.c_in / 8);
    const bool unit_w = pb.stride_w == 1 && pb.dil_w == 1;
    static PerDevice a3, a5, a0;
    cudaError_t e;
    if (dw_tma_eligible(pb)) return launch_dw_tma(pb, x, w, bias, z, st);
    const bool unit = unit_w && pb.stride_h == 1 && pb.dil_h == 1 && pb.kh == pb.kw && pb.pad_h >= 0 && pb.pad_w >= 0;
    if (unit && (pb.kh == 3 || pb.kh == 5)) {
        // rows per thread: as tall as still leaves every SM a few blocks
        int th = 8;
        auto threads = [&](int t) {
            return (long long)pb.n * ((pb.h_out + t - 1) / t) * ((pb.w_out + 1) / 2) * (pb.c_in / 8);
        };
        while (th > 1 && threads(th) < (long long)device_sm_count() * 256 * 4) th /= 2;
        static PerDevice s3, s5;
        if (pb.kh == 3) {
            auto threads4 = [&](int t) {
                return (long long)pb.n * ((pb.h_out + t - 1) / t) * ((pb.w_out + 1) / 2) * (pb.c_in / 4);
            };
            th = 16;
            while (th > 1 && threads4(th) < (long long)device_sm_count() * 256 * 4) th /= 2;
            if ((e = set_smem_once(dw_stream4_kernel<2, 3, 3>, &s3)) != cudaSuccess) return e;
            dw_stream4_kernel<2, 3, 3><<<dw_grid(threads4(th)), 256, smem, st>>>(s, (const uint2 *)x, (const __nv_bfloat16 *)w,
                                                                                bias, (uint2 *)z, th);
        } else {
            if ((e = set_smem_once(dw_stream_kernel<2, 5, 5>, &s5)) != cudaSuccess) return e;
            dw_stream_kernel<2, 5, 5><<<dw_grid(threads(th)), 256, smem, st>>>(s, (const uint4 *)x, (const __nv_bfloat16 *)w,
                                                                              bias, (uint4 *)z, th);
        }
    } else if (unit_w && pb.kw == 3) {
        if ((e = set_smem_once(dw_fwd_kernel<4, 3>, &a3)) != cudaSuccess) return e;
        dw_fwd_kernel<4, 3><<<dw_grid(total), 256, smem, st>>>(s, (const uint4 *)x, (const __nv_bfloat16 *)w, bias,
                                                                (uint4 *)z);
    } else if (unit_w && pb.kw == 5) {
        if ((e = set_smem_once(dw_fwd_kernel<4, 5>, &a5)) != cudaSuccess) return e;
        dw_fwd_kernel<4, 5><<<dw_grid(total), 256, smem, st>>>(s, (const uint4 *)x, (const __nv_bfloat16 *)w, bias,
                                                                (uint4 *)z);
    } else {
        if ((e = set_smem_once(dw_fwd_kernel<4, 0>, &a0)) != cudaSuccess) return e;
        dw_fwd_kernel<4, 0><<<dw_grid(total), 256, smem, st>>>(s, (const uint4 *)x, (const __nv_bfloat16 *)w, bias,
                                                                (uint4 *)z);
    }
    return cudaGetLastError();
}

cudaError_t launch_dw_dgrad(const Problem &pb, const void *dz, const void *w, void *dx, cudaStream_t st) {
    const DwShape s = dw_shape(pb);
    const size_t smem = (size_t)pb.kh * pb.kw * pb.c_in * sizeof(float);
    static PerDevice attr;
    cudaError_t e = set_smem_once(dw_dgrad_kernel, &attr);
    if (e != cudaSuccess) return e;
    const long long total = pb.pin * (pb.c_in / 8);
    dw_dgrad_kernel<<<dw_grid(total), 256, smem, st>>>(s, (const uint4 *)dz, (const __nv_bfloat16 *)w, (uint4 *)dx);
    return cudaGetLastError();
}

int dw_wgrad_splits(const Problem &pb) {
    long long want = (long long)device_sm_count() * 8;
    const long long cap = (pb.p + 63) / 64;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    const long long per = (pb.p + want - 1) / want;
    return (int)((pb.p + per - 1) / per);
}

template <int TAPS>
static cudaError_t launch_dw_wgrad_t(const Problem &pb, const void *dz, const void *x, float *part, int splits,
                                     cudaStream_t st) {
    const DwShape s = dw_shape(pb);
    const int v = pb.c_in / 8;
    const int block = (256 / v) * v;
    const size_t smem = (size_t)block * 8 * sizeof(float);
    const long long per = (pb.p + splits - 1) / splits;
    dw_wgrad_kernel<TAPS><<<splits, block, smem, st>>>(s, (const uint4 *)dz, (const uint4 *)x, part, (uint32_t)per);
    return cudaGetLastError();
}

bool dw_wgrad_supported(const Problem &pb) {
    const int t = pb.kh * pb.kw;
    return t == 9 || t == 25 || t == 1;
}

cudaError_t launch_dw_wgrad(const Problem &pb, const void *dz, const void *x, float *part, int splits,
                            cudaStream_t st) {
    if (pb.kh == 3 && pb.kw == 3 && pb.stride_h == 1 && pb.stride_w == 1 && pb.dil_h == 1 && pb.dil_w == 1) {
        const DwShape s = dw_shape(pb);
        const int v = pb.c_in / 8, block = (256 / v) * v;
        const long long items = (long long)pb.n * pb.h_out * ((pb.w_out + 3) / 4);
        const long long per = (items + splits - 1) / splits;
        dw_wgrad_window_kernel<4, 3, 3><<<splits, block, (size_t)block * 8 * sizeof(float), st>>>(
            s, (const uint4 *)dz, (const uint4 *)x, part, (uint32_t)per);
        return cudaGetLastError();
    }
    switch (pb.kh * pb.kw) {
        case 1: return launch_dw_wgrad_t<1>(pb, dz, x, part, splits, st);
        case 9: return launch_dw_wgrad_t<9>(pb, dz, x, part, splits, st);
        case 25: return launch_dw_wgrad_t<25>(pb, dz, x, part, splits, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace convbn
