// Forward pass of a first-layer ("stem") convolution with very few input channels, stride 2 along W
// (e.g. 7x7 stride 2 on RGB):  Z = omega' (*) X + b'  (Sec. 3.1 / 3.3), on the sm_100a tensor cores with the
// im2col expansion done by the MMA's own operand addressing instead of by memory traffic.
//
// Input rows are kept in shared memory as zero-bordered rows of 4-channel pixels (8 bytes each).  For one
// filter row r the K values of output pixel wo are the kw x 4 values that start at padded pixel 2 wo: 16 wo
// bytes into the row.  A K-major operand WITHOUT swizzle addresses element (m, k) at
//     start + (m / 8) SBO + (m % 8) 16 + (k / 8) LBO + (k % 8) 2      bytes,
// so SBO = 128 and LBO = 16 give  start + 16 m + 2 k : the 128 rows of the A tile are 128 consecutive output
// pixels of one output row, overlapping windows of the same shared-memory row.  Each input row is loaded
// once per tile (kh / stride_h times overall) instead of once per tap, and K per filter row is 32 (kw <= 8
// taps x 4 channels; unused slots meet zero weights), i.e. kh x 2 MMAs of 128 x C_out x 16 per output row.
//
// Warps: 0-7 load input rows (16-byte global loads, repacked 3 -> 4 channels on the way), 8-11 issue MMAs
// (round-robin over output rows, disjoint accumulators), 12-23 drain accumulators: scale, shift, bf16,
// swizzled staging, TMA store.  Every CTA owns a contiguous range of output rows.  Every wait is bounded.
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kWinLoaders = 8, kWinIssuers = 4, kWinEpiGroups = 3;
constexpr int kWinEpiWarp0 = kWinLoaders + kWinIssuers;
constexpr int kWinThreads = 32 * (kWinEpiWarp0 + 4 * kWinEpiGroups);
constexpr int kWinMaxStrips = 3;
constexpr int kWinSlack = 2304;          // bytes readable past the last row of a patch (junk rows of an M block)

struct WinGemm {
    int n, h_in, w_in, c_in, h_out, w_out, c_out, kh, kw, stride_h, pad_h, pad_w;
    int R;                 // output rows per tile
    int rows_in;           // input rows per full tile: (R - 1) stride_h + kh
    int pitch;             // bytes per padded input row in shared memory (multiple of 16)
    int colblocks;         // M blocks per output row: ceil(w_out / 128)
    int nstrips;           // patch buffers
    uint32_t strip_bytes;  // one patch buffer (multiple of 1024)
    int kblocks;           // 128-byte K rows of the resident weights: ceil(kh / 2)
    long long total_rows;  // n * h_out
    int f16;               // 16-bit storage type: 0 bf16, 1 IEEE half
    BnFold fold;
};

struct WinCtl {
    uint64_t strip_full[kWinMaxStrips], strip_empty[kWinMaxStrips];
    uint64_t tmem_full[8], tmem_empty[8];
    uint32_t tmem_base;
    int abort_flag;
    unsigned short slot_of[256];   // weight element (r, q, c) -> (K block << 8) | position in the 64-wide K row
};

// descriptor halves of the un-swizzled K-major window operand: LBO 16 bytes, SBO 128 bytes
__device__ __forceinline__ uint32_t win_desc_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3FFFu) | (1u << 16); }
__device__ __forceinline__ uint32_t win_desc_hi() { return 8u | (1u << 14); }

// The chunk sequence of a CTA: its output rows [lo, hi) of the flattened (image, row) space, cut into
// tiles of at most R rows that do not cross an image.  Every role walks the same sequence.
struct WinChunk { int img, h0, rows; };
__device__ __forceinline__ bool win_next_chunk(long long &cur, long long hi, int h_out, int R, WinChunk &c) {
    if (cur >= hi) return false;
    const long long img = cur / h_out;
    const int h0 = (int)(cur - img * h_out);
    int rows = R;
    if (rows > h_out - h0) rows = h_out - h0;
    if ((long long)rows > hi - cur) rows = (int)(hi - cur);
    c.img = (int)img; c.h0 = h0; c.rows = rows;
    cur += rows;
    return true;
}

// Fills `count` rows of a patch buffer with input rows first, first + 1, ... of image img: pixels of C channels
// widened to 4 (8 bytes) behind a left border of pad_w pixels; rows outside the image are zero.  fill3 is the
// bit pattern of channel slot 3 (C <= 3 only): 0, or bf16 1.0 when the weight-gradient GEMM takes sum dZ from it
// (then the caller has also set it in the borders).  Called by nthreads threads with ids tid.
template <int C>
__device__ __forceinline__ void win_fill_patch(uint8_t *patch, const __nv_bfloat16 *__restrict__ x, int img, int first,
                                               int count, int h_in, int w_in, int pad_w, int pitch, int tid, int nthreads,
                                               uint32_t fill3) {
    const int chunks_w = w_in / 8, tasks = count * chunks_w;
    const uint32_t hi_fill = fill3 << 16;
#pragma unroll 4
    for (int t = tid; t < tasks; t += nthreads) {
        const int pr = t / chunks_w, j = t - pr * chunks_w, h = first + pr;
        uint2 *dst = (uint2 *)(patch + (size_t)pr * pitch + (size_t)(pad_w + 8 * j) * 8);
        if (h < 0 || h >= h_in) {
#pragma unroll
            for (int p = 0; p < 8; ++p) dst[p] = make_uint2(0, hi_fill);
            continue;
        }
        const uint4 *src = (const uint4 *)(x + (((size_t)img * h_in + h) * w_in + 8 * j) * C);
        unsigned short e[8 * C];
#pragma unroll
        for (int v = 0; v < C; ++v) {
            const uint4 q4 = __ldg(src + v);
            e[8 * v + 0] = (unsigned short)q4.x; e[8 * v + 1] = (unsigned short)(q4.x >> 16);
            e[8 * v + 2] = (unsigned short)q4.y; e[8 * v + 3] = (unsigned short)(q4.y >> 16);
            e[8 * v + 4] = (unsigned short)q4.z; e[8 * v + 5] = (unsigned short)(q4.z >> 16);
            e[8 * v + 6] = (unsigned short)q4.w; e[8 * v + 7] = (unsigned short)(q4.w >> 16);
        }
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const unsigned short c0 = e[p * C], c1 = C > 1 ? e[p * C + (C > 1 ? 1 : 0)] : (unsigned short)0;
            const unsigned short c2 = C > 2 ? e[p * C + (C > 2 ? 2 : 0)] : (unsigned short)0;
            const uint32_t w1 = C > 3 ? ((uint32_t)c2 | ((uint32_t)e[p * C + (C > 3 ? 3 : 0)] << 16)) : ((uint32_t)c2 | hi_fill);
            dst[p] = make_uint2((uint32_t)c0 | ((uint32_t)c1 << 16), w1);
        }
    }
}

template <int BN, int C>
__global__ void __launch_bounds__(kWinThreads) stem_window_fwd_kernel(const __grid_constant__ CUtensorMap tm_out,
                                                                     const WinGemm g,
                                                                     const __nv_bfloat16 *__restrict__ x,
                                                                     const __nv_bfloat16 *__restrict__ w,
                                                                     const float *__restrict__ bias, int *err) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int NA = 512 / BN;                           // accumulators in tensor memory
    uint8_t *strips = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *wres = strips + (size_t)g.nstrips * g.strip_bytes;          // [kblocks][BN][128 B], 128-byte swizzle
    uint8_t *staging = wres + (size_t)g.kblocks * BN * 128;              // per epilogue warp [32 rows][128 B]
    WinCtl *ctl = (WinCtl *)(staging + 4 * kWinEpiGroups * 4096);
    float *bias_s = (float *)(((uintptr_t)(ctl + 1) + 15) & ~(uintptr_t)15);
    float *scale_s = bias_s + BN;
    const bool fold = g.fold.gamma != nullptr;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &ctl->abort_flag;
    // this CTA's output rows
    const long long row_lo = g.total_rows * blockIdx.x / gridDim.x, row_hi = g.total_rows * (blockIdx.x + 1) / gridDim.x;

    if (warp < kWinLoaders) {
        if (threadIdx.x == 0) {
            CONVBN_TRACE_POINT(0);
            for (int s = 0; s < kWinMaxStrips; ++s) { mbar_init(&ctl->strip_full[s], 32 * kWinLoaders); mbar_init(&ctl->strip_empty[s], kWinIssuers); }
            for (int s = 0; s < 8; ++s) { mbar_init(&ctl->tmem_full[s], 1); mbar_init(&ctl->tmem_empty[s], 4); }
            ctl->abort_flag = 0;
            fence_barrier_init();
            prefetch_tensormap(&tm_out);
            __threadfence_block();
        }
        // zero the patch buffers once: borders and the slack behind the last row stay zero for good
        {
            uint4 *p = (uint4 *)strips;
            const int n16 = (int)((size_t)g.nstrips * g.strip_bytes / 16);
            for (int i = threadIdx.x; i < n16; i += 32 * kWinLoaders) p[i] = make_uint4(0, 0, 0, 0);
        }
        __threadfence_block();
        named_bar_sync(3, 32 * kWinLoaders);
        named_bar_arrive(1, kWinThreads);
    }
    if (warp == kWinLoaders) {
        tmem_alloc(&ctl->tmem_base, 512);
        tmem_relinquish();
    }
    pdl_wait();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(1);
    uint32_t tmem_base = 0;
    if (warp >= kWinLoaders) {
        if (warp >= kWinEpiWarp0) {
            const int nt = kWinThreads - 32 * kWinEpiWarp0, tid = (int)threadIdx.x - 32 * kWinEpiWarp0;
            if (fold) {
                // On-the-fly reparameterisation (Sec. 3.3 / 3.4); s multiplies the fp32 accumulator (Sec. 3.2.2)
                for (int c = tid; c < BN; c += nt) {
                    const float r = 1.0f / sqrtf(g.fold.var[c] + g.fold.eps);
                    const float sc = g.fold.gamma[c] * r;
                    const float bf = ((g.fold.b ? g.fold.b[c] : 0.f) - g.fold.mean[c]) * sc + g.fold.beta[c];
                    scale_s[c] = sc;
                    bias_s[c] = bf;
                    if (blockIdx.x == 0 && g.fold.vec3) {
                        g.fold.vec3[c] = sc; g.fold.vec3[BN + c] = bf; g.fold.vec3[2 * BN + c] = r;
                    }
                }
            } else {
                for (int c = tid; c < BN; c += nt) { bias_s[c] = bias ? bias[c] : 0.f; scale_s[c] = 1.f; }
            }
            // resident weights: K index = r 32 + q 4 + c, two filter rows per 128-byte row, zeros in unused slots.
            // Zero everything, then scatter the real entries (consecutive threads read consecutive elements; the
            // loads of a batch are issued together).
            {
                uint4 *z4 = (uint4 *)wres;
                for (int i = tid; i < g.kblocks * BN * 8; i += nt) z4[i] = make_uint4(0, 0, 0, 0);
            }
            const int rowlen = g.kh * g.kw * C, total = BN * rowlen;
            if (tid < rowlen) {                        // the only divisions of the set-up: once per weight-row position
                const int c = tid % C, t2 = tid / C, q = t2 % g.kw, r = t2 / g.kw;
                ctl->slot_of[tid] = (unsigned short)(((r >> 1) << 8) | ((r & 1) * 32 + q * 4 + c));
            }
            named_bar_sync(4, nt);
            // 16-byte loads (8 weights), all of a thread's loads issued before the first use; channel = e / rowlen
            // by a multiply with the rounded-up reciprocal (e < 2^15: exact or one too large, fixed up)
            const uint4 *wsrc = (const uint4 *)w;
            const uint32_t inv = (65536u + (uint32_t)rowlen - 1u) / (uint32_t)rowlen;
            const int n8 = total / 8;                  // BN is a multiple of 64, so total is a multiple of 8
            for (int base = tid; base < n8; base += 4 * nt) {
                uint4 val[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) val[k] = base + k * nt < n8 ? __ldg(wsrc + base + k * nt) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (base + k * nt >= n8) break;
                    const uint32_t wd[4] = {val[k].x, val[k].y, val[k].z, val[k].w};
#pragma unroll
                    for (int h = 0; h < 8; ++h) {
                        const int e = (base + k * nt) * 8 + h;
                        int co = (int)(((uint32_t)e * inv) >> 16);
                        int rem = e - co * rowlen;
                        if (rem < 0) { --co; rem += rowlen; }
                        const int sl = ctl->slot_of[rem], k64 = sl & 255, kb = sl >> 8;
                        *(unsigned short *)(wres + (size_t)kb * BN * 128 + co * 128 + ((((k64 >> 3) ^ (co & 7)) & 7) << 4) + (k64 & 7) * 2) =
                            (unsigned short)(wd[h >> 1] >> ((h & 1) * 16));
                    }
                }
            }
            fence_proxy_async_smem();
        }
        tc_fence_before_sync();
        named_bar_sync(1, kWinThreads);
        tc_fence_after_sync();
        pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
        tmem_base = ctl->tmem_base;
        if (threadIdx.x == 32 * kWinLoaders) CONVBN_TRACE_POINT(2);
    }

    if (warp < kWinLoaders) {
        // ---------------- input-row loaders ----------------
        const int ltid = threadIdx.x;
        long long cur = row_lo;
        WinChunk ck;
        int sb = 0;
        uint32_t ph = 0;
        bool ok = true;
        while (ok && win_next_chunk(cur, row_hi, g.h_out, g.R, ck)) {
            { CONVBN_TRACE_T0();
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->strip_empty[sb], ph ^ 1u, abort_flag));
            if (threadIdx.x == 0) CONVBN_TRACE_ACC(12); }
            if (!ok) break;
            win_fill_patch<C>(strips + (size_t)sb * g.strip_bytes, x, ck.img, ck.h0 * g.stride_h - g.pad_h,
                              (ck.rows - 1) * g.stride_h + g.kh, g.h_in, g.w_in, g.pad_w, g.pitch, ltid, 32 * kWinLoaders, 0);
            fence_proxy_async_smem();                  // the tensor core reads these rows through the async proxy
            mbar_arrive(&ctl->strip_full[sb]);
            if (threadIdx.x == 0) { if (sb == 0 && ph == 0) CONVBN_TRACE_POINT(3); CONVBN_TRACE_POINT(8); }
            if (++sb == g.nstrips) { sb = 0; ph ^= 1u; }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    } else if (warp < kWinEpiWarp0) {
        // ---------------- MMA issuers: unit u (one M block = 128 output pixels of one row) goes to issuer u % 4
        const int me = warp - kWinLoaders;
        if (elect_one()) {
            const uint32_t idesc = idesc_h16_f32(128, BN, 0, 0, g.f16);
            const uint32_t a_hi = win_desc_hi(), b_hi = smem_desc_hi_sw128(1024);
            const uint32_t wres_lo = smem_desc_lo(smem_u32(wres), 16);
            long long cur = row_lo;
            WinChunk ck;
            int sb = 0;
            uint32_t sph = 0, u = 0;
            bool ok = true;
            while (ok && win_next_chunk(cur, row_hi, g.h_out, g.R, ck)) {
                const uint32_t patch_lo = win_desc_lo(smem_u32(strips + (size_t)sb * g.strip_bytes));
                bool have_patch = false;
                for (int i = 0; i < ck.rows && ok; ++i)
                    for (int cb = 0; cb < g.colblocks; ++cb, ++u) {
                        if ((int)(u % kWinIssuers) != me) continue;
                        if (!have_patch) {
                            { CONVBN_TRACE_T0();
                            if (!mbar_wait_bounded(&ctl->strip_full[sb], sph, abort_flag)) { ok = false; break; }
                            if (me == 0) CONVBN_TRACE_ACC(13); }
                            tc_fence_after_sync();
                            if (me == 0 && u == 0) CONVBN_TRACE_POINT(4);
                            have_patch = true;
                        }
                        const uint32_t slot = u % NA, use = u / NA;
                        { CONVBN_TRACE_T0();
                        if (!mbar_wait_bounded(&ctl->tmem_empty[slot], (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                        if (me == 0) CONVBN_TRACE_ACC(14); }
                        tc_fence_after_sync();
                        const uint32_t d = tmem_base + slot * BN;
                        // A: padded row (i stride_h + r), window start = pixel 2 (128 cb) -> 16 bytes per output pixel
                        uint32_t a_lo = patch_lo + (((uint32_t)(i * g.stride_h) * (uint32_t)g.pitch + (uint32_t)cb * 2048u) >> 4);
                        const uint32_t pitch16 = (uint32_t)g.pitch >> 4;
                        for (int r = 0; r < g.kh; ++r, a_lo += pitch16) {
                            const uint32_t b_lo = wres_lo + (uint32_t)(r >> 1) * (uint32_t)(BN * 128 >> 4) + (uint32_t)(r & 1) * 4u;
                            if (r == 0) umma_bf16_ss_halves<false>(d, a_lo, a_hi, b_lo, b_hi, idesc);
                            else umma_bf16_ss_halves<true>(d, a_lo, a_hi, b_lo, b_hi, idesc);
                            umma_bf16_ss_halves<true>(d, a_lo + 2u, a_hi, b_lo + 2u, b_hi, idesc);
                        }
                        umma_commit(&ctl->tmem_full[slot]);
                    }
                // this issuer's share of the patch is read once its MMAs complete (arrives at once if it had none)
                if (ok) umma_commit(&ctl->strip_empty[sb]);
                if (me == 0) { if (sb == 0 && sph == 0) CONVBN_TRACE_POINT(5); CONVBN_TRACE_POINT(6); }
                if (++sb == g.nstrips) { sb = 0; sph ^= 1u; }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else {
        // ---------------- epilogue: unit u goes to warp group u % 4; tensor memory -> scale, shift -> bf16 ->
        // swizzled staging -> TMA store of [32 pixels][64 channels] (pixels beyond the row end are clipped)
        const int quarter = warp & 3, egroup = (warp - kWinEpiWarp0) >> 2;
        uint8_t *buf = staging + (size_t)(warp - kWinEpiWarp0) * 4096;
        long long cur = row_lo;
        WinChunk ck;
        uint32_t u = 0;
        bool ok = true;
        while (ok && win_next_chunk(cur, row_hi, g.h_out, g.R, ck)) {
            for (int i = 0; i < ck.rows && ok; ++i)
                for (int cb = 0; cb < g.colblocks; ++cb, ++u) {
                    if ((int)(u % kWinEpiGroups) != egroup) continue;
                    const uint32_t slot = u % NA, use = u / NA;
                    { CONVBN_TRACE_T0();
                    ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->tmem_full[slot], use & 1u, abort_flag));
                    if (warp == kWinEpiWarp0 && lane == 0) CONVBN_TRACE_ACC(15); }
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int wo0 = cb * 128 + quarter * 32;
                    const int out_row = ck.img * g.h_out + ck.h0 + i;
                    const uint32_t t_row = tmem_base + slot * BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
                    for (int c0 = 0; c0 < BN; c0 += 64) {
                        const bool live = wo0 < g.w_out;           // else the whole box lies beyond the row end
                        if (live) {
                            if (lane == 0) tma_store_wait_read<0>();   // the previous store no longer reads the buffer
                            __syncwarp();
                        }
                        uint8_t *row = buf + lane * 128;
#pragma unroll 1
                        for (int half = 0; half < 2; ++half) {
                            uint32_t v[32];
                            if (live) {
                                tmem_ld_32x32(t_row + (uint32_t)(c0 + 32 * half), v);
                                tmem_ld_wait();
                            }
                            if (half == 1 && c0 + 64 >= BN) {
                                // every column of this accumulator has been read: hand it back
                                tc_fence_before_sync();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&ctl->tmem_empty[slot]);
                            }
                            if (!live) continue;
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                const int c = c0 + 32 * half + j;
                                const float4 s0 = *(const float4 *)(scale_s + c), s1 = *(const float4 *)(scale_s + c + 4);
                                const float4 b0 = *(const float4 *)(bias_s + c), b1 = *(const float4 *)(bias_s + c + 4);
                                uint4 pk;
                                pk.x = pack2_h16(fmaf(__uint_as_float(v[j]), s0.x, b0.x), fmaf(__uint_as_float(v[j + 1]), s0.y, b0.y), g.f16);
                                pk.y = pack2_h16(fmaf(__uint_as_float(v[j + 2]), s0.z, b0.z), fmaf(__uint_as_float(v[j + 3]), s0.w, b0.w), g.f16);
                                pk.z = pack2_h16(fmaf(__uint_as_float(v[j + 4]), s1.x, b1.x), fmaf(__uint_as_float(v[j + 5]), s1.y, b1.y), g.f16);
                                pk.w = pack2_h16(fmaf(__uint_as_float(v[j + 6]), s1.z, b1.z), fmaf(__uint_as_float(v[j + 7]), s1.w, b1.w), g.f16);
                                *(uint4 *)(row + (((4 * half + (j >> 3)) ^ (lane & 7)) << 4)) = pk;
                            }
                        }
                        if (!live) continue;
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_3d(&tm_out, buf, c0, wo0, out_row);
                            tma_store_commit();
                        }
                    }
                }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        if (warp == kWinEpiWarp0 && lane == 0) CONVBN_TRACE_POINT(9);
        if (lane == 0) tma_store_wait_all<0>();             // global writes done before the CTA exits
        if (warp == kWinEpiWarp0 && lane == 0) CONVBN_TRACE_POINT(10);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(11);
    if (warp == kWinLoaders) tmem_dealloc(ctl->tmem_base, 512);
}

// ---- weight gradient of the same layers ---------------------------------------------------------------
// domega'[co][r][q][c] = sum over images and output pixels of dZ[ho][wo][co] X[2 ho + r][2 wo + q][c]  (Sec. 3.2.1;
// Table 2, Tune row), with the same zero-bordered 4-channel rows in shared memory.  The contraction runs along the
// output pixels of a row (K = 16 pixels per MMA).  The M side is dZ: a row [wo][co] in 128-byte-swizzled rows is an
// MN-major operand of 64 rows (the channels), and two consecutive output rows of the chunk's dZ buffer make the
// 128 rows of one MMA.  The N side is the window of one input row, MN-major without swizzle: element (n, k) with
// n = 4 q + c and k = wo sits at  start + 2 n + 16 k, so 32 columns are the taps q = 0 .. 7 of all four channel
// slots.  Input row 2 ho + r is tap row r of output row ho and tap row r - 2 of output row ho + 1: with the
// accumulators of parity class e = r & 1 laid out as column blocks j of 32, lanes 0 - 63 of block j hold tap
// r = e + 2 j (from the even rows of the chunk) and lanes 64 - 127 hold tap r = e + 2 (j - 1) (from the odd rows),
// so ONE MMA serves both rows.  Block T_e of the lower lanes and block 0 of the upper lanes collect products that
// belong to no tap and are never read.  Channel slot 3 of every padded pixel holds 1.0 (C <= 3), so column n = 3
// of tap 0 is sum dZ.  Each CTA accumulates its contiguous range of output rows in tensor memory, adds the two
// lane halves through shared memory and writes one fp32 partial [k][co] plus one row of sums; the fused epilogue
// kernel adds the CTAs' partials in fixed order.
constexpr int kWgR = 4;                  // output rows per chunk
constexpr int kWgLoaders = 8;            // (a multiple of 4: the warps behind them own lane quarters 0, 1, 2, 3 of tensor memory in turn)
constexpr int kWgMovers = 4;             // one warp per lane quarter
// warps 0-7 X loaders, 8 tensor memory, 9 dZ producer, 10-11 issuers (8-11 read out), 12-15 dZ rows into tensor memory
constexpr int kWgThreads = 32 * (kWgLoaders + 4 + kWgMovers);
constexpr int kWgAccCols = 320;          // accumulators: two parity classes x (4 + 1) blocks of 32 columns
constexpr int kWgMaxSlots = 4;           // ring of dZ row pairs in the remaining 192 columns

struct WinWgrad {
    int n, h_in, w_in, h_out, w_out, c_out, kh, kw, pad_h, pad_w;
    int pitch, ksteps, T0, T1, kdim;
    int nslots;            // dZ row pairs that fit tensor memory beside the accumulators (8 ksteps columns each)
    uint32_t xstrip_bytes, dzrow_bytes;
    uint32_t work_bytes;   // operand buffers, at least the size of the read-out's exchange area
    long long total_rows;
    int f16;               // 16-bit storage type: 0 bf16, 1 IEEE half
};

struct WinWgCtl {
    uint64_t x_full[2], x_empty[2], dz_full[2], dz_empty[2], a_full[kWgMaxSlots], a_empty[kWgMaxSlots], acc_done;
    uint32_t tmem_base;
    int abort_flag;
};

template <int C>
__global__ void __launch_bounds__(kWgThreads) stem_window_wgrad_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                                      const WinWgrad g,
                                                                      const __nv_bfloat16 *__restrict__ x,
                                                                      float *__restrict__ partials,
                                                                      float *__restrict__ bsum,
                                                                      unsigned int *__restrict__ counters, int ncounters,
                                                                      int *err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *xs = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *dzs = xs + 2 * (size_t)g.xstrip_bytes;
    const uint32_t dzstrip = kWgR * g.dzrow_bytes;
    uint8_t *zeros = xs + g.work_bytes;                        // 16 zero rows of 128 bytes
    WinWgCtl *ctl = (WinWgCtl *)(zeros + 2048);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &ctl->abort_flag;
    const long long row_lo = g.total_rows * blockIdx.x / gridDim.x, row_hi = g.total_rows * (blockIdx.x + 1) / gridDim.x;

    if (threadIdx.x == 0) {
        CONVBN_TRACE_POINT(0);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&ctl->x_full[s], 32 * kWgLoaders); mbar_init(&ctl->x_empty[s], 2);
            mbar_init(&ctl->dz_full[s], 1); mbar_init(&ctl->dz_empty[s], kWgMovers);
        }
        for (int s = 0; s < kWgMaxSlots; ++s) { mbar_init(&ctl->a_full[s], kWgMovers); mbar_init(&ctl->a_empty[s], 2); }
        mbar_init(&ctl->acc_done, 2);
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_dz);
    }
    // every padded pixel starts as (0, 0, 0, 1): borders, rows outside the image and the slack keep that
    {
        uint4 *p4 = (uint4 *)xs;
        const int n16 = (int)(2 * (size_t)g.xstrip_bytes / 16);
        for (int i = threadIdx.x; i < n16; i += kWgThreads) p4[i] = make_uint4(0, one_h16(g.f16) << 16, 0, one_h16(g.f16) << 16);
        uint4 *z4 = (uint4 *)zeros;
        for (int i = threadIdx.x; i < 128; i += kWgThreads) z4[i] = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    if (warp == kWgLoaders) {
        tmem_alloc(&ctl->tmem_base, 512);
        tmem_relinquish();
    }
    pdl_wait();
    if (counters && blockIdx.x == 0)
        for (int i = threadIdx.x; i < ncounters; i += kWgThreads) counters[i] = 0u;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
    const uint32_t tmem_base = ctl->tmem_base;
    const uint32_t slot_cols = 8u * (uint32_t)g.ksteps;        // one dZ row pair: 8 columns per 16 pixels
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(1);

    if (warp < kWgLoaders) {
        // ---------------- X row loaders ----------------
        long long cur = row_lo;
        WinChunk ck;
        int sb = 0;
        uint32_t ph = 0;
        bool ok = true;
        while (ok && win_next_chunk(cur, row_hi, g.h_out, kWgR, ck)) {
            CONVBN_TRACE_T0();
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->x_empty[sb], ph ^ 1u, abort_flag));
            if (threadIdx.x == 0) CONVBN_TRACE_ACC(12);
            if (!ok) break;
            win_fill_patch<C>(xs + (size_t)sb * g.xstrip_bytes, x, ck.img, ck.h0 * 2 - g.pad_h, (ck.rows - 1) * 2 + g.kh,
                              g.h_in, g.w_in, g.pad_w, g.pitch, (int)threadIdx.x, 32 * kWgLoaders, one_h16(g.f16));
            fence_proxy_async_smem();
            mbar_arrive(&ctl->x_full[sb]);
            if (threadIdx.x == 0 && cur - ck.rows <= row_lo) CONVBN_TRACE_POINT(6);
            if (++sb == 2) { sb = 0; ph ^= 1u; }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    } else if (warp == kWgLoaders + 1) {
        // ---------------- dZ producer: one TMA box per output row of the chunk ----------------
        if (elect_one()) {
            long long cur = row_lo;
            WinChunk ck;
            int sb = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            while (ok && win_next_chunk(cur, row_hi, g.h_out, kWgR, ck)) {
                if (!mbar_wait_bounded(&ctl->dz_empty[sb], ph ^ 1u, abort_flag)) { ok = false; break; }
                mbar_arrive_expect_tx(&ctl->dz_full[sb], (uint32_t)ck.rows * g.dzrow_bytes);
                for (int i = 0; i < ck.rows; ++i)
                    tma_load_3d(dzs + (size_t)sb * dzstrip + (size_t)i * g.dzrow_bytes, &tm_dz, &ctl->dz_full[sb], 0, 0,
                                ck.img * g.h_out + ck.h0 + i);
                ++issued;
                if (++sb == 2) { sb = 0; ph ^= 1u; }
            }
            if (!ok) {
                atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1;
                // let the copies already issued land (bounded) before the CTA may exit
                for (int j = issued > 2 ? issued - 2 : 0; j < issued; ++j)
                    mbar_wait_bounded(&ctl->dz_full[j & 1], (uint32_t)(j >> 1) & 1u, nullptr, 200000000ull);
            }
        }
    } else if (warp >= kWgLoaders + 4) {
        // ---------------- dZ rows into tensor memory: the M side of the MMAs.  Lane m of a pair's tile is channel m & 63 of
        // the pair's row m >> 6; 16 pixels are 8 columns of two 16-bit elements.  (Read from tensor memory, the tile costs
        // the MMAs no shared-memory bandwidth: every pair meets up to 2 (T + 1) input rows.) ----------------
        const int q4 = (warp - (kWgLoaders + 4)) & 3, group = (warp - (kWgLoaders + 4)) >> 2;
        const int m = 32 * q4 + lane, half = m >> 6, co = m & 63;
        const uint32_t t_lane = tmem_base + ((uint32_t)(32 * q4) << 16) + (uint32_t)kWgAccCols;
        const uint32_t in_row = (uint32_t)(co & 7) * 2u;       // byte of the channel inside its 16-byte chunk
        long long cur = row_lo;
        WinChunk ck;
        int sb = 0, slot = 0;
        uint32_t ph = 0, aph = 0;
        bool ok = true;
        while (ok && win_next_chunk(cur, row_hi, g.h_out, kWgR, ck)) {
            { CONVBN_TRACE_T0();
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->dz_full[sb], ph, abort_flag));
            if (q4 == 0 && group == 0 && lane == 0) CONVBN_TRACE_ACC(15); }
            if (!ok) break;
            for (int i = 0; i < ck.rows; i += 2) {
                { CONVBN_TRACE_T0();
                ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->a_empty[slot], aph ^ 1u, abort_flag));
                if (q4 == 0 && group == 0 && lane == 0) CONVBN_TRACE_ACC(10); }
                if (!ok) break;
                tc_fence_after_sync();
                const bool have = i + half < ck.rows;           // an odd last pair has no second row: zeros
                const uint8_t *rowb = dzs + (size_t)sb * dzstrip + (size_t)(have ? i + half : 0) * g.dzrow_bytes;
                const uint32_t t0 = t_lane + (uint32_t)slot * slot_cols;
                for (int k = group; k < g.ksteps; k += kWgMovers / 4) {
                    uint32_t v[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        // pixels 16 k + 2 c and the next one; rows are 128-byte swizzled: chunk (co / 8) ^ (pixel & 7)
                        const uint32_t p0 = (uint32_t)(16 * k + 2 * c);
                        const uint32_t lo = *(const uint16_t *)(rowb + p0 * 128u + ((((uint32_t)(co >> 3) ^ (p0 & 7u)) & 7u) << 4) + in_row);
                        const uint32_t hi = *(const uint16_t *)(rowb + (p0 + 1u) * 128u + ((((uint32_t)(co >> 3) ^ ((p0 + 1u) & 7u)) & 7u) << 4) + in_row);
                        v[c] = have ? (lo | (hi << 16)) : 0u;
                    }
                    tmem_st_32x32_x8(t0 + 8u * (uint32_t)k, v);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->a_full[slot]);
                if (++slot == g.nslots) { slot = 0; aph ^= 1u; }
            }
            if (!ok) break;
            __syncwarp();                                       // the chunk's rows are in tensor memory: the buffer may be refilled
            if (lane == 0) mbar_arrive(&ctl->dz_empty[sb]);
            if (++sb == 2) { sb = 0; ph ^= 1u; }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    } else if (warp >= kWgLoaders + 2) {
        // ---------------- MMA issuers: one warp for the even input rows of a patch, one for the odd ones ----------------
        const int e = warp - (kWgLoaders + 2), Te = e ? g.T1 : g.T0;
        if (elect_one()) {
            const uint32_t acc = tmem_base + (uint32_t)e * (kWgAccCols / 2);
            // window (N side): MN-major, no swizzle: 8 elements per 16 bytes, next 8 elements 16 bytes on, next 8 pixels 128 bytes on
            const uint32_t w_hi = (16u >> 4) | (1u << 14), w_lbo = (128u >> 4) << 16;
            // all accumulator columns of this class start from zero: one MMA with 128 zero rows (shared memory, block stride 0) on the M side
            umma_bf16_ss_halves<false>(acc, smem_desc_lo(smem_u32(zeros), 0), smem_desc_hi_sw128(1024),
                                       ((smem_u32(xs) >> 4) & 0x3FFFu) | w_lbo, w_hi, idesc_h16_f32(128, 32 * (Te + 1), 1, 1, g.f16));
            const uint32_t idesc = idesc_h16_f32(128, 32, 0, 1, g.f16);       // M side in tensor memory (K-major), window MN-major
            long long cur = row_lo;
            WinChunk ck;
            int sb = 0, slot = 0;
            uint32_t ph = 0, aph = 0;
            bool ok = true;
            while (ok && win_next_chunk(cur, row_hi, g.h_out, kWgR, ck)) {
                CONVBN_TRACE_T0();
                if (!mbar_wait_bounded(&ctl->x_full[sb], ph, abort_flag)) { ok = false; break; }
                if (e == 0) CONVBN_TRACE_ACC(13);
                const uint32_t xa = smem_u32(xs + (size_t)sb * g.xstrip_bytes);
                const int count = (ck.rows - 1) * 2 + g.kh;
                for (int i = 0; i < ck.rows; i += 2) {
                    if (!mbar_wait_bounded(&ctl->a_full[slot], aph, abort_flag)) { ok = false; break; }
                    if (e == 0) CONVBN_TRACE_ACC(14);          // (x and dZ together)
                    if (e == 0 && i == 0 && cur - ck.rows <= row_lo) CONVBN_TRACE_POINT(2);
                    tc_fence_after_sync();
                    const uint32_t a0 = tmem_base + (uint32_t)kWgAccCols + (uint32_t)slot * slot_cols;
                    for (int pr = e; pr < count; pr += 2) {
                        const int t = ((pr - e) >> 1) - i;    // input row pr is tap row e + 2 t of output row i and e + 2 (t - 1) of row i + 1
                        const bool lower = t >= 0 && t < Te, upper = i + 1 < ck.rows && t >= 1 && t <= Te;
                        if (!lower && !upper) continue;
                        const uint32_t d = acc + 32u * (uint32_t)t;
                        uint32_t w_lo = (((xa + (uint32_t)pr * (uint32_t)g.pitch) >> 4) & 0x3FFFu) | w_lbo;
                        for (int k = 0; k < g.ksteps; ++k, w_lo += 16u)     // 16 pixels: 256 bytes of window, 8 columns of dZ
                            umma_h16_ts_acc(d, a0 + 8u * (uint32_t)k, w_lo, w_hi, idesc);
                    }
                    umma_commit(&ctl->a_empty[slot]);
                    if (++slot == g.nslots) { slot = 0; aph ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&ctl->x_empty[sb]);
                if (++sb == 2) { sb = 0; ph ^= 1u; }
            }
            if (e == 0) CONVBN_TRACE_POINT(3);
            if (ok) umma_commit(&ctl->acc_done);
            else { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    }
    // ---------------- read-out: warps 8 - 11 own lanes 0-31, 32-63, 64-95, 96-127 of tensor memory (lane = output channel,
    // lower half from the even rows of the chunks, upper half from the odd rows).  The halves are added through shared
    // memory: the lower warps hand over their odd tap rows and finish the even ones, the upper warps the reverse ----------------
    const int rw = warp - kWgLoaders;
    const bool reader = rw >= 0 && rw < 4;
    float *ex = (float *)xs;                   // exchange area [tap][n][co]: the operand buffers are free once acc_done is complete
    const bool up_half = rw >= 2;
    const int co = (rw & 1) * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)((reader ? rw : 0) * 32) << 16);
    bool rd_ok = false;
    if (reader) {
        rd_ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->acc_done, 0, abort_flag));
        if (!rd_ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        if (rw == 0 && lane == 0) CONVBN_TRACE_POINT(4);
        if (rd_ok) {
            tc_fence_after_sync();
            const int e = up_half ? 0 : 1, Te = e ? g.T1 : g.T0;       // the class this half gives away
            for (int t = 0; t < Te; ++t) {         // the upper lanes keep tap t in column block t + 1
                uint32_t v[32];
                tmem_ld_32x32(t_lane + (uint32_t)(e * (kWgAccCols / 2) + 32 * (t + (up_half ? 1 : 0))), v);
                tmem_ld_wait();
                float *dst = ex + (size_t)((e ? g.T0 : 0) + t) * (32 * 64) + co;
#pragma unroll
                for (int n = 0; n < 32; ++n) dst[n * 64] = __uint_as_float(v[n]);
            }
        }
    }
    __syncthreads();                           // every warp: the halves that were given away are in the exchange area
    if (reader && rd_ok && !*abort_flag) {
        const int e = up_half ? 1 : 0, Te = e ? g.T1 : g.T0;           // the class this half finishes
        float *prow = partials + (size_t)blockIdx.x * g.kdim * 64 + co;
        for (int t = 0; t < Te; ++t) {
            const int r = e + 2 * t;
            uint32_t v[32];
            tmem_ld_32x32(t_lane + (uint32_t)(e * (kWgAccCols / 2) + 32 * (t + (up_half ? 1 : 0))), v);
            tmem_ld_wait();
            const float *other = ex + (size_t)((e ? g.T0 : 0) + t) * (32 * 64) + co;
#pragma unroll
            for (int n = 0; n < 32; ++n) {
                const int q = n >> 2, c = n & 3;
                const float sum = __uint_as_float(v[n]) + other[n * 64];
                if (q < g.kw && c < C) prow[(size_t)((r * g.kw + q) * C + c) * 64] = sum;
                else if (C < 4 && r == 0 && n == 3) bsum[(size_t)blockIdx.x * 64 + co] = sum;      // sum dZ
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(5);
    if (warp == kWgLoaders) tmem_dealloc(tmem_base, 512);
}

// ---- host side --------------------------------------------------------------------------------------
namespace {

struct WinPlan { bool ok = false; int R = 0, nstrips = 0, pitch = 0, kblocks = 0; uint32_t strip_bytes = 0; size_t smem = 0; };

WinPlan plan_window(const Problem &pb) {
    WinPlan pl;
    if (pb.groups != 1 || pb.c_in > 4 || pb.stride_w != 2 || pb.stride_h != 2 || pb.dil_h != 1 ||
        pb.dil_w != 1 || pb.kw > 8 || pb.kh > 16 || (pb.c_out != 64 && pb.c_out != 128) || pb.w_in % 8 ||
        pb.pad_w > 64 || pb.pad_h > 64 || pb.p >= (1LL << 30) || pb.pin >= (1LL << 30))
        return pl;
    pl.pitch = (int)(((size_t)(pb.w_in + 2 * pb.pad_w) * 8 + 15) / 16 * 16);
    pl.kblocks = (pb.kh + 1) / 2;
    const size_t fixed = 1024 + 4 * kWinEpiGroups * 4096 + sizeof(WinCtl) + 2 * (size_t)pb.c_out * sizeof(float) + 32 +
                         (size_t)pl.kblocks * pb.c_out * 128;
    const size_t budget = 226 * 1024;
    for (int r = pb.h_out < 8 ? pb.h_out : 8; r >= 1; --r) {
        const size_t rows_in = (size_t)(r - 1) * pb.stride_h + pb.kh;
        const size_t sbytes = (rows_in * pl.pitch + kWinSlack + 1023) / 1024 * 1024;
        if (fixed + 2 * sbytes > budget) continue;
        int ns = (int)((budget - fixed) / sbytes);
        if (ns > kWinMaxStrips) ns = kWinMaxStrips;
        pl.ok = true; pl.R = r; pl.nstrips = ns; pl.strip_bytes = (uint32_t)sbytes; pl.smem = fixed + (size_t)ns * sbytes;
        break;
    }
    return pl;
}

template <int BN, int C>
cudaError_t launch_window(const CUtensorMap &tout, const WinGemm &g, size_t smem, const void *x, const void *w,
                          const float *bias, int *err, cudaStream_t st) {
    static PerDevice attr, carve;
    if (cudaError_t e = max_dynamic_smem_once(stem_window_fwd_kernel<BN, C>, 227 * 1024, &attr); e != cudaSuccess) return e;
    prefer_max_shared_once(stem_window_fwd_kernel<BN, C>, &carve);
    const long long sms = device_sm_count();
    const unsigned grid = (unsigned)(g.total_rows < sms ? g.total_rows : sms);
    return launch_pdl(stem_window_fwd_kernel<BN, C>, dim3(grid), dim3(kWinThreads), smem, st, tout, g,
                      (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, bias, err);
}

template <int BN>
cudaError_t launch_window_c(int c_in, const CUtensorMap &tout, const WinGemm &g, size_t smem, const void *x,
                            const void *w, const float *bias, int *err, cudaStream_t st) {
    switch (c_in) {
        case 1: return launch_window<BN, 1>(tout, g, smem, x, w, bias, err, st);
        case 2: return launch_window<BN, 2>(tout, g, smem, x, w, bias, err, st);
        case 3: return launch_window<BN, 3>(tout, g, smem, x, w, bias, err, st);
        default: return launch_window<BN, 4>(tout, g, smem, x, w, bias, err, st);
    }
}

}  // namespace

bool stem_window_eligible(const Problem &pb) { return plan_window(pb).ok; }

namespace {
struct WinWgPlan { bool ok = false; int pitch = 0, ksteps = 0; uint32_t xstrip = 0, dzrow = 0, work = 0; size_t smem = 0; };
WinWgPlan plan_window_wgrad(const Problem &pb) {
    WinWgPlan pl;
    if (!plan_window(pb).ok || pb.c_in > 3 || pb.c_out != 64 || pb.kh < 2 || pb.kh > 8 || pb.w_out > 256) return pl;
    pl.pitch = (int)(((size_t)(pb.w_in + 2 * pb.pad_w) * 8 + 15) / 16 * 16);
    pl.ksteps = (pb.w_out + 15) / 16;
    pl.xstrip = (uint32_t)((((size_t)(kWgR - 1) * 2 + pb.kh) * pl.pitch + kWinSlack + 1023) / 1024 * 1024);
    pl.dzrow = (uint32_t)pl.ksteps * 16 * 128;
    pl.work = 2 * pl.xstrip + 2 * (uint32_t)kWgR * pl.dzrow;
    if (pl.work < (uint32_t)pb.kh * 8192u) pl.work = (uint32_t)pb.kh * 8192u;       // the read-out's exchange area: kh taps x 32 x 64 floats
    pl.smem = 1024 + (size_t)pl.work + 2048 + sizeof(WinWgCtl) + 64;
    pl.ok = pl.smem <= 226 * 1024;
    return pl;
}
}  // namespace

bool stem_window_wgrad_eligible(const Problem &pb) { return plan_window_wgrad(pb).ok; }

// (one function per channel count: the once-per-device flags must not be shared between the kernels)
template <int C>
static cudaError_t launch_window_wgrad(const CUtensorMap &tdz, const WinWgrad &g, size_t smem, unsigned grid, const void *x,
                                       float *partials, float *bsum, unsigned int *counters, int *err, cudaStream_t st) {
    static PerDevice attr, carve;
    if (cudaError_t e = max_dynamic_smem_once(stem_window_wgrad_kernel<C>, 227 * 1024, &attr); e != cudaSuccess) return e;
    prefer_max_shared_once(stem_window_wgrad_kernel<C>, &carve);
    return launch_pdl(stem_window_wgrad_kernel<C>, dim3(grid), dim3(kWgThreads), smem, st, tdz, g,
                      (const __nv_bfloat16 *)x, partials, bsum, counters, g.c_out / 32, err);
}

int stem_window_wgrad_ctas(const Problem &pb) {
    const long long rows = (long long)pb.n * pb.h_out, sms = device_sm_count();
    return (int)(rows < sms ? rows : sms);
}

cudaError_t launch_stem_window_wgrad(const Problem &pb, const void *dz, const void *x, float *partials, float *bsum,
                                     unsigned int *counters, cudaStream_t st) {
    const WinWgPlan pl = plan_window_wgrad(pb);
    if (!pl.ok) return cudaErrorInvalidValue;
    WinWgrad g;
    g.n = pb.n; g.h_in = pb.h_in; g.w_in = pb.w_in; g.h_out = pb.h_out; g.w_out = pb.w_out; g.c_out = pb.c_out;
    g.kh = pb.kh; g.kw = pb.kw; g.pad_h = pb.pad_h; g.pad_w = pb.pad_w; g.pitch = pl.pitch; g.ksteps = pl.ksteps;
    g.T0 = (pb.kh + 1) / 2; g.T1 = pb.kh / 2; g.kdim = pb.kdim; g.xstrip_bytes = pl.xstrip; g.dzrow_bytes = pl.dzrow; g.work_bytes = pl.work;
    g.nslots = (512 - kWgAccCols) / (8 * pl.ksteps);        // at least 1: w_out <= 256 gives ksteps <= 16
    if (g.nslots > kWgMaxSlots) g.nslots = kWgMaxSlots;
    g.total_rows = (long long)pb.n * pb.h_out;
    g.f16 = call_f16();
    CUtensorMap tdz;
    const unsigned long long dims[3] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                        (unsigned long long)pb.n * pb.h_out};
    const unsigned long long str[3] = {0, (unsigned long long)pb.c_out * 2, (unsigned long long)pb.w_out * pb.c_out * 2};
    const unsigned int box[3] = {64, (unsigned)pl.ksteps * 16, 1};
    if (!make_tmap_tiled_bf16(&tdz, dz, 3, dims, str, box)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)stem_window_wgrad_ctas(pb);
    switch (pb.c_in) {
        case 1: return launch_window_wgrad<1>(tdz, g, pl.smem, grid, x, partials, bsum, counters, err, st);
        case 2: return launch_window_wgrad<2>(tdz, g, pl.smem, grid, x, partials, bsum, counters, err, st);
        default: return launch_window_wgrad<3>(tdz, g, pl.smem, grid, x, partials, bsum, counters, err, st);
    }
}

cudaError_t launch_stem_window_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                                   cudaStream_t st, const BnFold *fold) {
    const WinPlan pl = plan_window(pb);
    if (!pl.ok) return cudaErrorInvalidValue;
    WinGemm g;
    g.n = pb.n; g.h_in = pb.h_in; g.w_in = pb.w_in; g.c_in = pb.c_in; g.h_out = pb.h_out; g.w_out = pb.w_out;
    g.c_out = pb.c_out; g.kh = pb.kh; g.kw = pb.kw; g.stride_h = pb.stride_h; g.pad_h = pb.pad_h; g.pad_w = pb.pad_w;
    g.R = pl.R; g.rows_in = (pl.R - 1) * pb.stride_h + pb.kh; g.pitch = pl.pitch;
    g.colblocks = (pb.w_out + 127) / 128; g.nstrips = pl.nstrips; g.strip_bytes = pl.strip_bytes;
    g.kblocks = pl.kblocks; g.total_rows = (long long)pb.n * pb.h_out;
    g.f16 = call_f16();
    g.fold = fold ? *fold : BnFold{nullptr, nullptr, nullptr, nullptr, nullptr, 0.f, nullptr};
    CUtensorMap tout;
    const unsigned long long dims[3] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                        (unsigned long long)pb.n * pb.h_out};
    const unsigned long long str[3] = {0, (unsigned long long)pb.c_out * 2, (unsigned long long)pb.w_out * pb.c_out * 2};
    const unsigned int box[3] = {64, 32, 1};
    if (!make_tmap_tiled_bf16(&tout, z, 3, dims, str, box)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    if (pb.c_out == 64) return launch_window_c<64>(pb.c_in, tout, g, pl.smem, x, w, bias, err, st);
    return launch_window_c<128>(pb.c_in, tout, g, pl.smem, x, w, bias, err, st);
}

}  // namespace convbn
