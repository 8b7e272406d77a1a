// First-layer ("stem") convolutions: very few input channels (C_in <= 8, e.g. 7x7 stride 2 on RGB).
// A pixel is then only 6-16 bytes, too narrow for TMA and for a 64-wide K block.  The input is first
// repacked to 8 channels per pixel (16 bytes) with an explicit zero border, after which the kw <= 8
// pixels a filter row touches are 128 contiguous bytes: one K row of 64 "channels" (8 pixels x 8
// channels) per filter row r.  A 5-D strided tensor map exposes those overlapping windows to TMA, and
// the dense tensor-core kernels run with K = kh * 64 (zeros in the unused slots of the weights).
// Stride-2 layers with at most 4 channels use a denser space-to-depth packing (see stem_s2d below).
#include "kernels.h"
#include "mma_sync.cuh"

namespace convbn {

bool stem_eligible(const Problem &pb) {
    return pb.groups == 1 && pb.c_in <= 8 && pb.kw <= 8 && pb.kh <= 16 && pb.dil_h == 1 && pb.dil_w == 1 &&
           pb.stride_h <= 4 && pb.stride_w <= 4 && pb.c_out % 64 == 0 && pb.c_out <= 1024 &&
           pb.p < (1LL << 30) && pb.pin < (1LL << 30);
}

// Stride-2 layers with C_in <= 4 are packed "space to depth" instead: a packed pixel holds the 2 x 2 block
// of padded input pixels (2 I + a, 2 J + b) as [a][b][4 channels] = 16 values (32 bytes).  Tap (r, q) of
// output (ho, wo) is then element (r & 1, q & 1) of packed pixel (ho + r / 2, wo + q / 2), and the four
// packed pixels wo .. wo + 3 of packed row ho + tr are 128 contiguous bytes: one K row of 64 per PAIR of
// filter rows, K = ceil(kh / 2) * 64 instead of kh * 64 (7 x 7: 256 instead of 448, 57 % of it real taps).
bool stem_s2d(const Problem &pb) { return pb.stride_h == 2 && pb.stride_w == 2 && pb.c_in <= 4; }

int stem_krows(const Problem &pb) { return stem_s2d(pb) ? (pb.kh + 1) / 2 : pb.kh; }

// With at most 3 channels the fourth channel slot of a packed pixel is free: the packing kernel writes the
// constant 1 into slot (a, b, c) = (0, 0, 3), where the forward weights are zero.  In the weight-gradient
// GEMM row 3 of the k rows is then sum_p dZ[p][co], and the separate slice of ones (a third of that
// kernel's CTAs for a 7 x 7 stem) is not needed.
bool stem_ones_in_pack(const Problem &pb) { return stem_s2d(pb) && pb.c_in <= 3; }

void stem_geometry(const Problem &pb, int *hp, int *wp) {
    if (stem_s2d(pb)) {
        const int need_h = (pb.h_out - 1) + stem_krows(pb), need_w = (pb.w_out - 1) + 4;
        const int have_h = (pb.h_in + 2 * pb.pad_h + 1) / 2, have_w = (pb.w_in + 2 * pb.pad_w + 1) / 2;
        *hp = need_h > have_h ? need_h : have_h;
        *wp = need_w > have_w ? need_w : have_w;
        return;
    }
    const int need_h = (pb.h_out - 1) * pb.stride_h + pb.kh, need_w = (pb.w_out - 1) * pb.stride_w + 8;
    const int have_h = pb.h_in + 2 * pb.pad_h, have_w = pb.w_in + 2 * pb.pad_w;
    *hp = need_h > have_h ? need_h : have_h;
    *wp = need_w > have_w ? need_w : have_w;
}

size_t stem_packed_bytes(const Problem &pb) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    return (size_t)pb.n * hp * wp * (stem_s2d(pb) ? 32 : 16);
}

void stem_window_strides(const Problem &pb, unsigned long long str[5]) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    if (stem_s2d(pb)) {      // one packed pixel per output column, one packed row per output row and per K row
        str[0] = 0; str[1] = 32; str[2] = (unsigned long long)wp * 32; str[3] = (unsigned long long)wp * 32;
        str[4] = (unsigned long long)hp * wp * 32;
    } else {
        str[0] = 0; str[1] = (unsigned long long)pb.stride_w * 16; str[2] = (unsigned long long)pb.stride_h * wp * 16;
        str[3] = (unsigned long long)wp * 16; str[4] = (unsigned long long)hp * wp * 16;
    }
}

size_t stem_weight_bytes(const Problem &pb) { return (size_t)pb.c_out * stem_krows(pb) * 64 * 2; }

// xp[n][hp][wp][a][b][4] = x[n][2 I + a - pad_h][2 J + b - pad_w][c] inside the image, 0 elsewhere
__global__ void __launch_bounds__(256) stem_pack_s2d_kernel(int n, int h_in, int w_in, int c_in, int pad_h, int pad_w,
                                                            int hp, int wp, int ones, int f16,
                                                            const __nv_bfloat16 *__restrict__ x,
                                                            uint4 *__restrict__ xp) {
    const long long total = (long long)n * hp * wp * 2;          // one thread per (packed pixel, a)
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int a = (int)(i & 1);
        const long long pix = i >> 1;
        const int wq = (int)(pix % wp);
        const long long t = pix / wp;
        const int hq = (int)(t % hp), img = (int)(t / hp);
        const int h = 2 * hq + a - pad_h;
        unsigned short v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (ones && a == 0) v[3] = (unsigned short)one_h16(f16);   // 1.0 in slot (0, 0, 3), border included
        if (h >= 0 && h < h_in) {
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const int w = 2 * wq + b - pad_w;
                if (w >= 0 && w < w_in) {
                    const unsigned short *src = (const unsigned short *)x + (((long long)img * h_in + h) * w_in + w) * c_in;
                    for (int c = 0; c < c_in; ++c) v[b * 4 + c] = src[c];
                }
            }
        }
        uint4 q;
        q.x = v[0] | ((uint32_t)v[1] << 16); q.y = v[2] | ((uint32_t)v[3] << 16);
        q.z = v[4] | ((uint32_t)v[5] << 16); q.w = v[6] | ((uint32_t)v[7] << 16);
        xp[i] = q;
    }
}

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
    const long long total = (long long)pb.n * hp * wp * (stem_s2d(pb) ? 2 : 1);
    long long blocks = (total + 255) / 256;
    if (blocks > device_sm_count() * 16) blocks = device_sm_count() * 16;
    if (stem_s2d(pb)) {
        stem_pack_s2d_kernel<<<(int)blocks, 256, 0, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.pad_h, pb.pad_w, hp, wp,
                                                          stem_ones_in_pack(pb) ? 1 : 0, call_f16(), (const __nv_bfloat16 *)x,
                                                          (uint4 *)xp);
        return cudaGetLastError();
    }
    stem_pack_kernel<<<(int)blocks, 256, 0, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.pad_h, pb.pad_w, hp, wp,
                                                  (const __nv_bfloat16 *)x, (uint4 *)xp);
    return cudaGetLastError();
}

// wst[co][r][q * 8 + c] = scale[co] * w[co][r][q][c]  (q < kw, c < C_in), zero elsewhere; space-to-depth
// packing (s2d): wst[co][tr][tq * 16 + a * 8 + b * 4 + c] with r = 2 tr + a, q = 2 tq + b
__global__ void __launch_bounds__(256) stem_expand_weights_kernel(int c_out, int kh, int kw, int c_in, int krows,
                                                                  int s2d, const __nv_bfloat16 *__restrict__ w,
                                                                  const float *__restrict__ s_vec,
                                                                  __nv_bfloat16 *__restrict__ wst, int f16) {
    const int total = c_out * krows * 64;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int j = i & 63, kr = (i >> 6) % krows, co = (i >> 6) / krows;
        const int r = s2d ? 2 * kr + ((j >> 3) & 1) : kr;
        const int q = s2d ? 2 * (j >> 4) + ((j >> 2) & 1) : j >> 3, c = s2d ? (j & 3) : (j & 7);
        float v = 0.f;
        if (r < kh && q < kw && c < c_in)
            v = (s_vec ? s_vec[co] : 1.f) * load_h16(w + (((long long)co * kh + r) * kw + q) * c_in + c, f16);
        reinterpret_cast<uint16_t *>(wst)[i] = pack1_h16(v, f16);
    }
}

cudaError_t launch_stem_expand_weights(const Problem &pb, const void *w, const float *s_vec, void *wst,
                                       cudaStream_t st) {
    const int total = pb.c_out * stem_krows(pb) * 64;
    stem_expand_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(pb.c_out, pb.kh, pb.kw, pb.c_in, stem_krows(pb),
                                                                    stem_s2d(pb) ? 1 : 0, (const __nv_bfloat16 *)w, s_vec,
                                                                    (__nv_bfloat16 *)wst, call_f16());
    return cudaGetLastError();
}

// ---- backward data of a stem layer ------------------------------------------------------------------
// dX[n,h,w,c] = sum over the taps that reach (h, w) and over co of omega'[co,r,q,c] dZ[n,ho,wo,co]
// (Sec. 3.2.1).  As a GEMM this has N = C_in <= 8 columns: too narrow for a 128-row tcgen05 tile (its
// smallest N is 16, and the A operand would stream through shared memory once per tap), so the kernel
// uses warp-level m16n8k16 MMAs with fp32 accumulation instead.  One MMA tile is 16 consecutive pixels
// of one row and one residue class (h mod stride_h, w mod stride_w), so that all of them meet the same
// taps; K runs over 64 output channels per tap.  The contraction order over the channels is free as
// long as A and B agree, which lets every lane fetch its A fragments with 16-byte loads straight from
// dZ: lane (g, t) reads 8-channel chunks t and t + 4 of pixels g and g + 8, and k-step k takes word k
// of each chunk.  The B fragments (the scaled weights, rounded to bf16) are laid out in shared memory
// in exactly that order, one 32-bit word per lane and fragment register.
// A warp owns 32 consecutive columns of one dZ row at a time (two MMA tiles).  With NU taps in a kernel
// row of the class, tap u pairs output pixel j with dZ column j + const - u, so instead of loading
// shifted A fragments per tap the warp keeps one accumulator per tap over the un-shifted columns and
// applies the shifts once at the end, through a small shared-memory scratch: every A fragment is
// loaded once per kernel row rather than once per tap, and 32 - (NU - 1) output pixels come out of
// each 32-column window.
template <int NU, bool H>      // NU: taps per kernel row and class, rounded up to 1, 2, 4 or 8; H: IEEE-half storage, else bf16
__global__ void __launch_bounds__(256) stem_dgrad_kernel(int n, int h_in, int w_in, int c_in, int h_out, int w_out,
                                                         int c_out, int kh, int kw, int stride_h, int stride_w,
                                                         int pad_h, int pad_w, const uint4 *__restrict__ dz,
                                                         const __nv_bfloat16 *__restrict__ w,
                                                         const float *__restrict__ s_vec,
                                                         __nv_bfloat16 *__restrict__ dx) {
    extern __shared__ uint32_t wfrag[];    // [tap][64-channel block][k-step][b0/b1][lane], then the scratch
    constexpr int OUTW = 32 - (NU - 1);    // output pixels per window
    const int taps = kh * kw;
    const int ncb = c_out / 64, v = c_out / 8;
#pragma unroll 4
    for (int i = threadIdx.x; i < taps * ncb * 256; i += blockDim.x) {
        const int t = i & 3, g = (i >> 2) & 7, which = (i >> 5) & 1, k = (i >> 6) & 3;
        const int cb = (i >> 8) % ncb, tap = (i >> 8) / ncb;
        const int co = cb * 64 + which * 32 + 8 * t + 2 * k;
        uint32_t word = 0u;
        if (g < c_in) {
            const float w0 = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((size_t)co * taps + tap) * c_in + g, H ? 1 : 0);
            const float w1 =
                (s_vec ? s_vec[co + 1] : 1.f) * load_h16(w + ((size_t)(co + 1) * taps + tap) * c_in + g, H ? 1 : 0);
            word = pack2_t<H>(w0, w1);
        }
        wfrag[i] = word;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    float *scr = reinterpret_cast<float *>(wfrag + (size_t)taps * ncb * 256) + warp * 256;   // [32 columns][8]
    const uint32_t wpb = blockDim.x >> 5;                      // windows per block and pass
    // Work items are (pass of wpb windows, residue class).  A block owns a contiguous run of passes and
    // visits every class of a pass before the next pass: the classes of one pass, and neighbouring
    // passes, read the same rows of dZ, and every block meets the classes equally often although they
    // have different tap counts.
    const int wt_max = ((w_in + stride_w - 1) / stride_w + OUTW - 1) / OUTW;
    const uint32_t ipc = ((uint32_t)n * ((h_in + stride_h - 1) / stride_h) * wt_max + wpb - 1) / wpb;
    const uint32_t ncls = (uint32_t)(stride_h * stride_w);
    const uint32_t run = (ipc + gridDim.x - 1) / gridDim.x;
    const uint32_t pass_end = min(ipc, (blockIdx.x + 1) * run);
    for (uint32_t item = blockIdx.x * run * ncls; item < pass_end * ncls; ++item) {
        const int cls = (int)(item % ncls);
        const int a = cls / stride_w, b = cls % stride_w;
        if (a >= h_in || b >= w_in) continue;
        const int hi_n = (h_in - a + stride_h - 1) / stride_h, wj_n = (w_in - b + stride_w - 1) / stride_w;
        const int wt_n = (wj_n + OUTW - 1) / OUTW;             // windows along a row
        const uint32_t idx = (item / ncls) * wpb + warp;
        if (idx >= (uint32_t)n * hi_n * wt_n) continue;        // whole warp
        const uint32_t t1 = idx / (uint32_t)wt_n;
        const int jbase = (int)(idx - t1 * (uint32_t)wt_n) * OUTW;
        const int img = (int)(t1 / (uint32_t)hi_n);
        const int h = (int)(t1 - (uint32_t)img * (uint32_t)hi_n) * stride_h + a;
        const int r0 = (a + pad_h) % stride_h, q0 = (b + pad_w) % stride_w;
        const int nu = q0 < kw ? (kw - q0 + stride_w - 1) / stride_w : 0;   // <= NU
        // tap u (q = q0 + u stride_w) pairs output pixel j with column j + (b + pad_w - q0) / stride_w - u;
        // window column p holds dZ column col0 + p, so tap u's product for pixel jbase + l sits at l + NU-1 - u
        const int col0 = jbase + (b + pad_w - q0) / stride_w - (NU - 1);
        float acc[NU][2][4];
#pragma unroll
        for (int u = 0; u < NU; ++u)
#pragma unroll
            for (int tl = 0; tl < 2; ++tl)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[u][tl][c] = 0.f;
        // this lane's four dZ columns of the window (tile 0 / 1, rows g / g + 8): validity and offset inside
        // a dZ row are the same for every kernel row, only the row changes
        bool col_ok[2][2];
        int col_off[2][2];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int wo = col0 + tl * 16 + g + 8 * hh;
                col_ok[tl][hh] = wo >= 0 && wo < w_out;
                col_off[tl][hh] = col_ok[tl][hh] ? wo * v + t : 0;
            }
        const uint4 *img_base = dz + (size_t)img * h_out * w_out * v;
        const int wstep = stride_w * ncb * 256;                // fragment words between two taps of a class
        for (int cb = 0; cb < ncb; ++cb) {
            for (int r = r0; r < kh; r += stride_h) {
                // h + pad_h - r is a multiple of the stride inside a class, also when negative
                const int ho = (h + pad_h - r) / stride_h;
                if (ho < 0 || ho >= h_out) continue;
                const uint4 *row = img_base + (size_t)ho * w_out * v + cb * 8;
                uint4 alo[2][2], ahi[2][2];                    // columns g / g + 8 of a tile, chunks t / t + 4
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int tl = 0; tl < 2; ++tl) {
                    alo[tl][0] = col_ok[tl][0] ? __ldg(row + col_off[tl][0]) : zero;
                    alo[tl][1] = col_ok[tl][0] ? __ldg(row + col_off[tl][0] + 4) : zero;
                    ahi[tl][0] = col_ok[tl][1] ? __ldg(row + col_off[tl][1]) : zero;
                    ahi[tl][1] = col_ok[tl][1] ? __ldg(row + col_off[tl][1] + 4) : zero;
                }
                const uint32_t *wf = wfrag + ((r * kw + q0) * ncb + cb) * 256 + lane;
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    if (u < nu) {                              // the same for the whole warp
                        uint32_t bf[4][2];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            bf[k][0] = wf[u * wstep + k * 64];
                            bf[k][1] = wf[u * wstep + k * 64 + 32];
                        }
#pragma unroll
                        for (int tl = 0; tl < 2; ++tl) {
                            mma_16x8x16_t<H>(acc[u][tl], alo[tl][0].x, ahi[tl][0].x, alo[tl][1].x, ahi[tl][1].x, bf[0][0], bf[0][1]);
                            mma_16x8x16_t<H>(acc[u][tl], alo[tl][0].y, ahi[tl][0].y, alo[tl][1].y, ahi[tl][1].y, bf[1][0], bf[1][1]);
                            mma_16x8x16_t<H>(acc[u][tl], alo[tl][0].z, ahi[tl][0].z, alo[tl][1].z, ahi[tl][1].z, bf[2][0], bf[2][1]);
                            mma_16x8x16_t<H>(acc[u][tl], alo[tl][0].w, ahi[tl][0].w, alo[tl][1].w, ahi[tl][1].w, bf[3][0], bf[3][1]);
                        }
                    }
                }
            }
        }
        // Shift and add: accumulator registers are (column g, channels 2t, 2t+1) and (column g + 8, same);
        // lane l then owns output pixel jbase + l with all 8 channels.
        float res[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) res[c] = 0.f;
#pragma unroll
        for (int u = 0; u < NU; ++u) {
            if (u < nu) {
                __syncwarp();
#pragma unroll
                for (int tl = 0; tl < 2; ++tl)
#pragma unroll
                    for (int half = 0; half < 2; ++half)
                        *reinterpret_cast<float2 *>(scr + (tl * 16 + g + 8 * half) * 8 + 2 * t) =
                            make_float2(acc[u][tl][2 * half], acc[u][tl][2 * half + 1]);
                __syncwarp();
                if (lane < OUTW) {
                    const float4 *src = reinterpret_cast<const float4 *>(scr + (lane + NU - 1 - u) * 8);
                    const float4 x0 = src[0], x1 = src[1];
                    res[0] += x0.x; res[1] += x0.y; res[2] += x0.z; res[3] += x0.w;
                    res[4] += x1.x; res[5] += x1.y; res[6] += x1.z; res[7] += x1.w;
                }
            }
        }
        const int j = jbase + lane;
        if (lane < OUTW && j < wj_n) {
            __nv_bfloat16 *dst = dx + ((size_t)(img * h_in + h) * w_in + j * stride_w + b) * c_in;
#pragma unroll
            for (int c = 0; c < 8; ++c)
                if (c < c_in) reinterpret_cast<uint16_t *>(dst)[c] = pack1_h16(res[c], H ? 1 : 0);
        }
    }
}

bool stem_dgrad_eligible(const Problem &pb) {
    return stem_eligible(pb) && (size_t)pb.kh * pb.kw * (pb.c_out / 64) * 1024 + 8192 <= 160 * 1024;
}

cudaError_t launch_stem_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                              cudaStream_t st) {
    const size_t smem = (size_t)pb.kh * pb.kw * (pb.c_out / 64) * 1024 + 8192;   // fragments + 1 KB per warp
    const int nu = (pb.kw + pb.stride_w - 1) / pb.stride_w;    // taps per kernel row in the fullest class
    const bool half = call_f16() != 0;
    const void *fns[2][4] = {{(const void *)stem_dgrad_kernel<1, false>, (const void *)stem_dgrad_kernel<2, false>,
                              (const void *)stem_dgrad_kernel<4, false>, (const void *)stem_dgrad_kernel<8, false>},
                             {(const void *)stem_dgrad_kernel<1, true>, (const void *)stem_dgrad_kernel<2, true>,
                              (const void *)stem_dgrad_kernel<4, true>, (const void *)stem_dgrad_kernel<8, true>}};
    static PerDevice attr;
    if (!attr.done[current_device_slot()]) {
        for (int h = 0; h < 2; ++h)
            for (int i = 0; i < 4; ++i)
                if (cudaError_t e = cudaFuncSetAttribute(fns[h][i], cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
                    e != cudaSuccess)
                    return e;
        attr.done[current_device_slot()] = true;
    }
    const void *fn = fns[half ? 1 : 0][nu <= 1 ? 0 : nu <= 2 ? 1 : nu <= 4 ? 2 : 3];
    int per_sm = 0, dev = 0, sms = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, 256, smem);
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    const long long passes = ((long long)pb.n * pb.h_in * pb.w_in + 255) / 256;
    const long long resident = (long long)per_sm * sms;        // one wave of persistent blocks
    const unsigned grid = (unsigned)(passes < resident ? passes : resident);
#define CONVBN_STEM_DGRAD(NU_, H_)                                                                                    \
    stem_dgrad_kernel<NU_, H_><<<grid, 256, smem, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.c_out, \
                                                        pb.kh, pb.kw, pb.stride_h, pb.stride_w, pb.pad_h, pb.pad_w,   \
                                                        (const uint4 *)dz, (const __nv_bfloat16 *)w, s_vec,           \
                                                        (__nv_bfloat16 *)dx)
    if (half) {
        if (nu <= 1) CONVBN_STEM_DGRAD(1, true);
        else if (nu <= 2) CONVBN_STEM_DGRAD(2, true);
        else if (nu <= 4) CONVBN_STEM_DGRAD(4, true);
        else CONVBN_STEM_DGRAD(8, true);
    } else {
        if (nu <= 1) CONVBN_STEM_DGRAD(1, false);
        else if (nu <= 2) CONVBN_STEM_DGRAD(2, false);
        else if (nu <= 4) CONVBN_STEM_DGRAD(4, false);
        else CONVBN_STEM_DGRAD(8, false);
    }
#undef CONVBN_STEM_DGRAD
    return cudaGetLastError();
}

}  // namespace convbn
