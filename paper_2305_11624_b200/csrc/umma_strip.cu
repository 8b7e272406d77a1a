// Stride-1 k x k convolution on the sm_100a tensor cores with the input staged ONCE per tile.
//
// The im2col kernel (umma_conv.cu) reloads every input pixel once per filter tap; for 3x3 layers that
// is 9x the input through L2 and the TMA ring's latency bounds the kernel.  Here a tile is R output
// rows x CW output columns of one image.  Its (R + kh - 1) x (CW + kw - 1) input patch is loaded by
// one tiled TMA copy per 64-channel chunk into shared memory as a flat list of pixels, 128 bytes
// each, 128-byte swizzled.  Number the tile's outputs, halo columns included, as "virtual pixels"
// v = i Wt + j (Wt = CW + kw - 1): tap (r, q) of virtual pixel v reads patch pixel v + r Wt + q, so the
// A operand of tap (r, q) for 128 consecutive virtual pixels is the SAME shared memory, read from a
// start address shifted by (r Wt + q) pixels.  All taps of a chunk are issued from one copy.
// Junk virtual pixels (j >= CW or i >= R) are computed and dropped.
//
//   forward        Z  = omega' (*) X + b'   (Sec. 3.1 / 3.3)   activation X,  weights omega'
//   backward data  dX = omega'_rot (*) dZ   (Sec. 3.2.1)       activation dZ, rotated / swapped omega'
//
// Warps: 0 patch loader (ring of 2-4 patch buffers), 1 weight-tile loader, 2-5 MMA issuers (warp 2 owns the
// tensor memory), 6-21 epilogue (four per tensor-memory lane quarter).  Every wait is bounded.
// One thread can issue a narrow MMA only every 60-100 clocks once the loop around it is counted, while a
// 128 x 64 x 16 MMA executes in 48: the M blocks of a tile are therefore dealt to up to four issuing warps,
// which write disjoint accumulators and each commit to the shared barriers (arrival count = issuers).
// The weight tiles either stream through a 4-slot ring, once per tile, or - when the whole matrix of the
// CTA's output channels fits beside the patch buffers - are loaded once and stay resident, which makes small
// tiles (more rounds over the SMs, better balance) free of weight traffic.
#include <string.h>

#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kSIssuers = 4;            // MMA-issuing warps (each owns a subset of a tile's M blocks)
constexpr int kSEpiGroups = 4;          // epilogue warps per tensor-memory lane quarter
constexpr int kSEpiWarp0 = 2 + kSIssuers;
constexpr int kSThreads = 32 * (kSEpiWarp0 + 4 * kSEpiGroups);   // 2 loader, 4 issuer and 16 epilogue warps
constexpr int kSBStages = 12;         // weight-tile ring: at most this many slots
constexpr int kSMaxStrips = 4;        // patch buffers
constexpr int kSMaxAcc = 4;           // accumulator sets (tiles in flight between the issuers and the epilogue)

struct StripGemm {
    int n, ho, wo, cn, ca, kh, kw, lower_h, lower_w;
    int R, CW, Wt, rows_in, nmb;      // tile rows / columns, patch width, patch rows, M blocks of 128
    int tiles_h, tiles_w;
    uint32_t strip_bytes;             // one patch buffer (multiple of 1024)
    int nacc;                         // accumulator sets in tensor memory (2 .. kSMaxAcc)
    int blockdiag;                    // grouped conv as block-diagonal 64-channel GEMMs: output block j reads input chunk j
    uint32_t tmem_cols;
    int nstrips;                      // patch buffers in the ring (2 .. kSMaxStrips)
    int bstages;                      // weight-tile ring slots in use (streaming mode)
    int nissue;                       // issuing warps in use: min(nmb, kSIssuers)
    int resident;                     // 1: all weight tiles stay in shared memory (one n-tile only)
    int f16;                          // 16-bit storage type: 0 bf16, 1 IEEE half
    int sub_cin, sub_hin, sub_win;    // sub-pixel output mode, see UmmaConvShape
    int sub_wide;                     // 1: wide sub-pixel mode (BN = 64 / 128), n-tile -> parity class
    uint32_t sub_mask[4];             // taps with weights, per class
    __nv_bfloat16 *out;
    BnFold fold;
};

struct StripCtl {
    uint64_t strip_full[kSMaxStrips], strip_empty[kSMaxStrips];
    uint64_t b_full[kSBStages], b_empty[kSBStages];
    uint64_t bres_full;               // resident weights have landed
    uint64_t tmem_full[kSMaxAcc], tmem_empty[kSMaxAcc];
    uint32_t tmem_base;
    int abort_flag;
};

// One stage of a 4 x 4 transpose inside a quad of lanes: the lane whose bit is set gives `lo` and takes the partner's
// `hi` in its place; the other lane gives `hi` and takes the partner's `lo`.
__device__ __forceinline__ void quad_swap(uint4 &lo, uint4 &hi, int mask, bool upper) {
    const uint4 send = upper ? lo : hi;
    uint4 recv;
    recv.x = __shfl_xor_sync(0xffffffffu, send.x, mask);
    recv.y = __shfl_xor_sync(0xffffffffu, send.y, mask);
    recv.z = __shfl_xor_sync(0xffffffffu, send.z, mask);
    recv.w = __shfl_xor_sync(0xffffffffu, send.w, mask);
    if (upper) lo = recv; else hi = recv;
}

template <int BN>
__global__ void __launch_bounds__(kSThreads) umma_strip_conv_kernel(const __grid_constant__ CUtensorMap tm_act,
                                                                   const __grid_constant__ CUtensorMap tm_w,
                                                                   const StripGemm g, const float *__restrict__ bias,
                                                                   int *err) {
    extern __shared__ uint8_t smem_raw[];
    constexpr uint32_t kBBytes = BN * 64 * 2;
    uint8_t *strips = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *bring = strips + (size_t)g.nstrips * g.strip_bytes;     // weight ring, or the resident weight tiles
    const int cchunks = g.blockdiag ? 1 : g.ca / 64, taps = g.kh * g.kw;
    const int bstages = g.bstages;
    StripCtl *ctl = (StripCtl *)(bring + (size_t)(g.resident ? taps * cchunks : bstages) * kBBytes);
    float *bias_s = (float *)(((uintptr_t)(ctl + 1) + 15) & ~(uintptr_t)15);
    float *scale_s = bias_s + g.cn;
    const bool fold = g.fold.gamma != nullptr;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstrips = g.nstrips;
    const int w_ca = g.blockdiag ? 64 : g.ca;          // K extent of one tap in the weight matrix
    const uint32_t n_tiles = (uint32_t)g.cn / BN;
    const uint32_t sp_tiles = (uint32_t)g.n * g.tiles_h * g.tiles_w;
    const uint32_t total_tiles = sp_tiles * n_tiles;
    volatile int *abort_flag = &ctl->abort_flag;

    // Set-up.  Warp 0 (thread 0) initialises the barriers and goes straight to its loads; warp 1 waits only
    // for that (named barrier 2); the other warps allocate tensor memory and form the per-channel scale and
    // shift, and meet on named barrier 1, on which the two loader warps merely arrive.  The first patch and
    // the first weight tiles are therefore in flight while the rest of the set-up runs.
    if (warp == 0) {
        if (lane == 0) {
            CONVBN_TRACE_POINT(0);
            const uint32_t ni = (uint32_t)g.nissue;     // every issuer commits to the barriers its MMAs release
            for (int s = 0; s < kSMaxStrips; ++s) { mbar_init(&ctl->strip_full[s], 1); mbar_init(&ctl->strip_empty[s], ni); }
            for (int s = 0; s < kSMaxAcc; ++s) { mbar_init(&ctl->tmem_full[s], ni); mbar_init(&ctl->tmem_empty[s], 4 * kSEpiGroups); }
            for (int s = 0; s < kSBStages; ++s) { mbar_init(&ctl->b_full[s], 1); mbar_init(&ctl->b_empty[s], ni); }
            mbar_init(&ctl->bres_full, 1);
            ctl->abort_flag = 0;
            fence_barrier_init();
            // the tensor maps are kernel parameters, not data of an earlier kernel: fetch them before the wait
            prefetch_tensormap(&tm_act); prefetch_tensormap(&tm_w);
            __threadfence_block();
        }
        __syncwarp();
        named_bar_arrive(2, 64);
        named_bar_arrive(1, kSThreads);
    } else if (warp == 1) {
        named_bar_sync(2, 64);
        named_bar_arrive(1, kSThreads);
    }
    if (warp == 2) {
        tmem_alloc(&ctl->tmem_base, g.tmem_cols);
        tmem_relinquish();
    }
    // Everything above touched only this CTA's own shared / tensor memory.  Global memory (inputs that an
    // earlier kernel may still be writing, outputs it may still be reading) comes after this wait.
    pdl_wait();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(1);
    uint32_t tmem_base = 0;
    if (warp >= 2) {
        const int nt = kSThreads - 64, tid = (int)threadIdx.x - 64;
        if (fold) {
            // On-the-fly reparameterisation (Sec. 3.3 / 3.4): s = gamma / sqrt(var + eps), b' = (b - mu) s + beta;
            // s multiplies the fp32 accumulator (the associative law of Sec. 3.2.2), so omega is used unrounded.
            for (int c = tid; c < g.cn; c += nt) {
                const float r = 1.0f / sqrtf(g.fold.var[c] + g.fold.eps);
                const float sc = g.fold.gamma[c] * r;
                const float bf = ((g.fold.b ? g.fold.b[c] : 0.f) - g.fold.mean[c]) * sc + g.fold.beta[c];
                scale_s[c] = sc;
                bias_s[c] = bf;
                if (blockIdx.x == 0 && g.fold.vec3) {
                    g.fold.vec3[c] = sc; g.fold.vec3[g.cn + c] = bf; g.fold.vec3[2 * g.cn + c] = r;
                }
            }
        } else if (bias) {
            for (int c = tid; c < g.cn; c += nt) bias_s[c] = bias[c];
        }
        tc_fence_before_sync();
        named_bar_sync(1, kSThreads);
        tc_fence_after_sync();
        pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
        tmem_base = ctl->tmem_base;
        if (threadIdx.x == 64) CONVBN_TRACE_POINT(2);
    }

    // tile t -> (image, tile row, tile column, n-tile); n-tiles of one patch sit on neighbouring CTAs
    auto decode = [&](uint32_t t, int &img, int &h0, int &w0, int &n0) {
        const uint32_t sp = t / n_tiles;
        n0 = (int)(t - sp * n_tiles) * BN;
        const uint32_t a = sp / (uint32_t)g.tiles_w;
        w0 = (int)(sp - a * (uint32_t)g.tiles_w) * g.CW;
        const uint32_t b = a / (uint32_t)g.tiles_h;
        h0 = (int)(a - b * (uint32_t)g.tiles_h) * g.R;
        img = (int)b;
    };

    if (warp == 0) {
        // ---------------- patch loader: one TMA copy per (tile, channel chunk) ----------------
        if (elect_one()) {
            int sb = 0;
            uint32_t ph = 0;
            const uint32_t bytes = (uint32_t)g.rows_in * g.Wt * 128u;
            bool ok = true;
            for (uint32_t t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                int img, h0, w0, n0;
                decode(t, img, h0, w0, n0);
                for (int cc = 0; cc < cchunks; ++cc) {
                    if (!mbar_wait_bounded(&ctl->strip_empty[sb], ph ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(&ctl->strip_full[sb], bytes);
                    if (t == blockIdx.x && cc == 0) CONVBN_TRACE_POINT(3);
                    tma_load_4d(strips + (size_t)sb * g.strip_bytes, &tm_act, &ctl->strip_full[sb],
                                g.blockdiag ? n0 : cc * 64, w0 + g.lower_w, h0 + g.lower_h, img);
                    if (++sb == nstrips) { sb = 0; ph ^= 1u; }
                }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
            // an issued copy always completes; give the last ones time to land before the CTA can exit
            if (!ok) for (int s = 0; s < nstrips; ++s) mbar_wait_bounded(&ctl->strip_full[s], 0, nullptr, 2000000ull);
        }
    } else if (warp == 1) {
        // ---------------- weight-tile loader ----------------
        if (elect_one()) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (g.resident) {
                // one n-tile, every (channel chunk, tap) tile loaded once: tile index cc taps + tap
                if (blockIdx.x < total_tiles) {
                    mbar_arrive_expect_tx(&ctl->bres_full, (uint32_t)(taps * cchunks) * kBBytes);
                    for (int cc = 0; cc < cchunks; ++cc)
                        for (int tap = 0; tap < taps; ++tap)
                            tma_load_2d(bring + (size_t)(cc * taps + tap) * kBBytes, &tm_w, &ctl->bres_full,
                                        tap * w_ca + cc * 64, 0);
                }
            } else
            for (uint32_t t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const int n0 = (int)(t % n_tiles) * BN;
                const uint32_t mask = g.sub_wide ? g.sub_mask[n0 / g.sub_cin] : 0xffffffffu;
                for (int cc = 0; cc < cchunks && ok; ++cc)
                    for (int tap = 0; tap < taps; ++tap) {
                        if (!((mask >> tap) & 1u)) continue;
                        if (!mbar_wait_bounded(&ctl->b_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                        mbar_arrive_expect_tx(&ctl->b_full[s], kBBytes);
                        tma_load_2d(bring + (size_t)s * kBBytes, &tm_w, &ctl->b_full[s], tap * w_ca + cc * 64, n0);
                        if (++s == bstages) { s = 0; ph ^= 1u; }
                    }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
            if (!ok) for (int q = 0; q < bstages; ++q) mbar_wait_bounded(&ctl->b_full[q], 0, nullptr, 2000000ull);
        }
    } else if (warp < kSEpiWarp0) {
        // ---------------- MMA issuers ----------------
        // One thread issues every MMA, so the instructions between two MMAs bound the rate of the narrow
        // ones (a 128 x 64 x 16 MMA takes 48 clocks, a 128 x 16 x 16 one 39): descriptors are kept as halves
        // and only their start-address field moves.
        const int me = warp - 2, ni = g.nissue;         // this warp issues M blocks me, me + ni, ...
        if (me < ni && elect_one()) {
            const uint32_t idesc = idesc_h16_f32(128, BN, 0, 0, g.f16);
            const uint32_t hi = smem_desc_hi_sw128(1024);
            const uint32_t bres_lo = smem_desc_lo(smem_u32(bring), 16);
            int sb = 0, s = 0;
            uint32_t sph = 0, bph = 0, i = 0;
            bool ok = true;
            if (g.resident && blockIdx.x < total_tiles) {
                ok = mbar_wait_bounded(&ctl->bres_full, 0, abort_flag);
                tc_fence_after_sync();
            }
            for (uint32_t t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++i) {
                const uint32_t a = i % (uint32_t)g.nacc, use = i / (uint32_t)g.nacc;
                if (!mbar_wait_bounded(&ctl->tmem_empty[a], (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d0 = tmem_base + a * (uint32_t)(g.nmb * BN);
                const uint32_t mask = g.sub_wide ? g.sub_mask[(int)(t % n_tiles) * BN / g.sub_cin] : 0xffffffffu;
                bool started = false;                   // false until the tile's first MMAs have been issued
                for (int cc = 0; cc < cchunks && ok; ++cc) {
                    if (!mbar_wait_bounded(&ctl->strip_full[sb], sph, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (i == 0 && cc == 0 && me == 0) CONVBN_TRACE_POINT(4);
                    const uint32_t a_patch = smem_desc_lo(smem_u32(strips + (size_t)sb * g.strip_bytes), 16);
                    uint32_t row_shift = 0;             // (r Wt + q) pixels of 128 bytes, in 16-byte units
                    int q = 0;
                    for (int tap = 0; tap < taps; ++tap) {
                        const uint32_t a_tap = a_patch + row_shift + (uint32_t)q * 8u;
                        if (++q == g.kw) { q = 0; row_shift += (uint32_t)g.Wt * 8u; }
                        if (!((mask >> tap) & 1u)) continue;
                        uint32_t b_lo;
                        if (g.resident) {
                            b_lo = bres_lo + (uint32_t)(cc * taps + tap) * (kBBytes >> 4);
                        } else {
                            if (!mbar_wait_bounded(&ctl->b_full[s], bph, abort_flag)) { ok = false; break; }
                            tc_fence_after_sync();
                            b_lo = smem_desc_lo(smem_u32(bring + (size_t)s * kBBytes), 16);
                        }
                        // consecutive MMAs go to different accumulators (M blocks), so an MMA never has to
                        // wait for the previous one's accumulator update
                        if (!started) {
                            for (int mb = me; mb < g.nmb; mb += ni)
                                umma_bf16_ss_halves<false>(d0 + (uint32_t)(mb * BN), a_tap + (uint32_t)mb * 1024u, hi, b_lo, hi, idesc);
                            started = true;
                        } else {
                            for (int mb = me; mb < g.nmb; mb += ni)
                                umma_bf16_ss_halves<true>(d0 + (uint32_t)(mb * BN), a_tap + (uint32_t)mb * 1024u, hi, b_lo, hi, idesc);
                        }
#pragma unroll
                        for (int k = 1; k < 4; ++k)
                            for (int mb = me; mb < g.nmb; mb += ni)
                                umma_bf16_ss_halves<true>(d0 + (uint32_t)(mb * BN), a_tap + (uint32_t)mb * 1024u + (uint32_t)k * 2u, hi,
                                                          b_lo + (uint32_t)k * 2u, hi, idesc);
                        if (!g.resident) {
                            umma_commit(&ctl->b_empty[s]);
                            if (++s == bstages) { s = 0; bph ^= 1u; }
                        }
                    }
                    if (ok) umma_commit(&ctl->strip_empty[sb]);
                    if (++sb == nstrips) { sb = 0; sph ^= 1u; }
                }
                if (ok) umma_commit(&ctl->tmem_full[a]);
                if (me == 0) { if (i == 0) CONVBN_TRACE_POINT(5); CONVBN_TRACE_POINT(6); }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else {
        // ---------------- epilogue: tensor memory -> registers -> (scale, shift) -> bf16 -> global ----
        const int quarter = warp & 3;
        const int egroup = (warp - kSEpiWarp0) >> 2;   // M blocks egroup, egroup + 4, ... of every tile
        uint32_t i = 0;
        for (uint32_t t = blockIdx.x; t < total_tiles; t += gridDim.x, ++i) {
            const uint32_t a = i % (uint32_t)g.nacc, use = i / (uint32_t)g.nacc;
            const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->tmem_full[a], use & 1u, abort_flag));
            if (!ok) {
                if (lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
                break;
            }
            tc_fence_after_sync();
            if (warp == kSEpiWarp0 && lane == 0) { if (i == 0) CONVBN_TRACE_POINT(7); CONVBN_TRACE_POINT(9); }
            int img, h0, w0, n0;
            decode(t, img, h0, w0, n0);
            for (int mb = egroup; mb < g.nmb; mb += kSEpiGroups) {
                const uint32_t v = (uint32_t)mb * 128u + (uint32_t)(quarter * 32 + lane);
                const uint32_t vi = v / (uint32_t)g.Wt;
                const int ti = (int)vi, tj = (int)(v - vi * (uint32_t)g.Wt);
                const int h = h0 + ti, wq = w0 + tj;
                const bool valid = ti < g.R && tj < g.CW && h < g.ho && wq < g.wo;
                __nv_bfloat16 *orow = g.out + ((size_t)((size_t)img * g.ho + (valid ? h : 0)) * g.wo + (valid ? wq : 0)) * g.cn + n0;
                bool store = valid;
                if (BN != 16 && g.sub_wide) {
                    // this n-tile holds channels [c_off, c_off + BN) of input position (2 h + a2, 2 wq + b2)
                    const int cls = n0 / g.sub_cin, c_off = n0 - cls * g.sub_cin;
                    const int hh = 2 * h + (cls >> 1), ww = 2 * wq + (cls & 1);
                    store = valid && hh < g.sub_hin && ww < g.sub_win;
                    orow = g.out + (((size_t)img * g.sub_hin + (store ? hh : 0)) * g.sub_win + (store ? ww : 0)) * g.sub_cin + c_off;
                }
                const uint32_t t_row = tmem_base + (a * (uint32_t)g.nmb + (uint32_t)mb) * BN + ((uint32_t)(quarter * 32) << 16);
                if constexpr (BN == 16) {
                    // sub-pixel mode: columns 8 a2 + e (e = b cin + ci) go to input row 2 h + a2, elements
                    // e of the 2 cin consecutive values that start at column 2 wq
                    uint32_t vv[16];
                    tmem_ld_32x16(t_row, vv);
                    tmem_ld_wait();
                    if (valid) {
                        const int cin = g.sub_cin;
                        int lim = (g.sub_win - 2 * wq) * cin;          // elements left in the row
                        if (lim > 2 * cin) lim = 2 * cin;
                        const bool pairs = ((g.sub_win * cin) & 1) == 0;   // every row start is 4-byte aligned
#pragma unroll
                        for (int a2 = 0; a2 < 2; ++a2) {
                            const int hh = 2 * h + a2;
                            if (hh < g.sub_hin) {
                                __nv_bfloat16 *dst = g.out + (((size_t)img * g.sub_hin + hh) * g.sub_win + (size_t)(2 * wq)) * cin;
#pragma unroll
                                for (int e = 0; e < 8; e += 2) {
                                    const float f0 = __uint_as_float(vv[a2 * 8 + e]), f1 = __uint_as_float(vv[a2 * 8 + e + 1]);
                                    if (pairs && e + 1 < lim) {
                                        *(uint32_t *)(dst + e) = pack2_h16(f0, f1, g.f16);
                                    } else {
                                        if (e < lim) reinterpret_cast<uint16_t *>(dst)[e] = pack1_h16(f0, g.f16);
                                        if (e + 1 < lim) reinterpret_cast<uint16_t *>(dst)[e + 1] = pack1_h16(f1, g.f16);
                                    }
                                }
                            }
                        }
                    }
                } else {
                // A lane holds one pixel's row of the accumulator; 32 lanes storing 16 bytes each, 2 BN bytes apart,
                // would touch 32 lines per instruction.  The four lanes of a quad transpose their 4 x 4 blocks of
                // 16-byte chunks instead, so that every store instruction writes 64 contiguous bytes per quad.
                const int quad0 = lane & ~3, qc = lane & 3;
                const unsigned long long optr = (unsigned long long)(uintptr_t)orow;
                __nv_bfloat16 *rowp[4];
                bool rowok[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const unsigned long long pk64 = __shfl_sync(0xffffffffu, optr, quad0 + k);
                    rowp[k] = (__nv_bfloat16 *)(uintptr_t)pk64;
                    rowok[k] = __shfl_sync(0xffffffffu, (int)store, quad0 + k) != 0;
                }
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t vv[32];
                    tmem_ld_32x32(t_row + (uint32_t)c0, vv);
                    tmem_ld_wait();
                    uint4 pk[4];
                    auto pack_chunk = [&](auto half_tag) {
                        constexpr bool H = decltype(half_tag)::value;
    #pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            float f[8];
    #pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(vv[j + e]);
                            if (fold) {
                                const float4 s0 = *(const float4 *)(scale_s + n0 + c0 + j);
                                const float4 s1 = *(const float4 *)(scale_s + n0 + c0 + j + 4);
                                f[0] *= s0.x; f[1] *= s0.y; f[2] *= s0.z; f[3] *= s0.w;
                                f[4] *= s1.x; f[5] *= s1.y; f[6] *= s1.z; f[7] *= s1.w;
                            }
                            if (bias || fold) {
                                const float4 b0 = *(const float4 *)(bias_s + n0 + c0 + j);
                                const float4 b1 = *(const float4 *)(bias_s + n0 + c0 + j + 4);
                                f[0] += b0.x; f[1] += b0.y; f[2] += b0.z; f[3] += b0.w;
                                f[4] += b1.x; f[5] += b1.y; f[6] += b1.z; f[7] += b1.w;
                            }
                            pk[j >> 3].x = pack2_t<H>(f[0], f[1]);
                            pk[j >> 3].y = pack2_t<H>(f[2], f[3]);
                            pk[j >> 3].z = pack2_t<H>(f[4], f[5]);
                            pk[j >> 3].w = pack2_t<H>(f[6], f[7]);
                        }
                    };
                    if (g.f16) pack_chunk(std::true_type{}); else pack_chunk(std::false_type{});
                    // butterfly transpose: afterwards pk[k] of lane (quad0 + c) is chunk c of row (quad0 + k)
                    quad_swap(pk[0], pk[1], 1, (lane & 1) != 0);
                    quad_swap(pk[2], pk[3], 1, (lane & 1) != 0);
                    quad_swap(pk[0], pk[2], 2, (lane & 2) != 0);
                    quad_swap(pk[1], pk[3], 2, (lane & 2) != 0);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (rowok[k]) *(uint4 *)(rowp[k] + c0 + qc * 8) = pk[k];
                }
                }
            }
            // this warp has read all it needs from the accumulator set
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->tmem_empty[a]);
            if (warp == kSEpiWarp0 && lane == 0) { if (i == 0) CONVBN_TRACE_POINT(8); CONVBN_TRACE_POINT(10); }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(11);
    if (warp == 2) tmem_dealloc(tmem_base, g.tmem_cols);
}

// ---- host side --------------------------------------------------------------------------------------
namespace {

struct StripPlan { bool ok = false; int bn = 64, R = 0, CW = 0, Wt = 0, nmb = 0, nacc = 2, tiles_w = 1 << 20, nstrips = 2, resident = 0, bstages = 4; uint32_t strip_bytes = 0; size_t smem = 0; };

int strip_sm_count() { return device_sm_count(); }

StripPlan plan_strip_search(const UmmaConvShape &s);

// The search below runs a double loop over tile shapes and is asked for several times per library call
// (eligibility, workspace size, launch): its result is cached per thread, keyed by the shape and the SM count.
StripPlan plan_strip(const UmmaConvShape &s) {
    struct Entry { UmmaConvShape key; int sms; StripPlan plan; bool used; };
    thread_local Entry cache[16] = {};
    thread_local int next = 0;
    const int sms = strip_sm_count();
    for (const Entry &e : cache)
        if (e.used && e.sms == sms && memcmp(&e.key, &s, sizeof(UmmaConvShape)) == 0) return e.plan;
    Entry &slot = cache[next];
    next = (next + 1) % 16;
    memcpy(&slot.key, &s, sizeof(UmmaConvShape));
    slot.sms = sms;
    slot.plan = plan_strip_search(s);
    slot.used = true;
    return slot.plan;
}

StripPlan plan_strip_search(const UmmaConvShape &s) {
    StripPlan best;
    if (s.stride_h != 1 || s.stride_w != 1 || s.dil_h != 1 || s.dil_w != 1 || s.out_sw) return best;
    if (s.blockdiag && s.ca != s.cn) return best;
    const bool sub = s.sub_cin > 0 && s.cn == 16, sub_wide = s.sub_cin > 0 && !sub;
    if (s.sub_cin > 0 && s.blockdiag) return best;
    if (sub_wide && (s.sub_cin % 64 || s.cn != 4 * s.sub_cin)) return best;
    if (s.taps_h * s.taps_w < 2 || s.ca % 64 || (!sub && s.cn % 64) || s.cn > 4096 || s.wo < 14 || s.ho < 2) return best;
    if ((long long)s.n * s.ho * s.wo >= (1LL << 30)) return best;
    // wide sub-pixel mode: an n-tile must not straddle two parity classes
    const int bn = sub ? 16 : (sub_wide ? (s.sub_cin % 128 == 0 ? 128 : 64) : ((s.cn % 128 == 0 && !s.blockdiag) ? 128 : 64));
    const int nmb_max = 512 / bn / 2;                      // two accumulator sets
    const int tiles_w_min = (s.wo + (256 - s.taps_w + 1) - 1) / (256 - s.taps_w + 1);
    // Among the tilings that keep at least 70 % of the MMA rows useful, take the one with the lowest
    // estimated time: rounds over the SMs x (the larger of the tile's MMA issue time and its shared-memory
    // fill time, plus a fixed cost per tile).  Weight tiles that do not stay resident are streamed again for
    // every tile, so small tiles then pay for them many times over.
    const int cchunks = s.blockdiag ? 1 : s.ca / 64, taps = s.taps_h * s.taps_w;
    const int n_tiles = s.cn / bn, sms = strip_sm_count();
    const size_t fixed = 1024 + sizeof(StripCtl) + 2 * (size_t)s.cn * sizeof(float) + 32;
    const size_t bbytes = (size_t)bn * 128, wall = (size_t)taps * cchunks * bbytes;
    const size_t budget = 224 * 1024;
    // clocks per 128 x bn x 16 MMA (measured issue floors 39 / 48 / 64, plus the issue loop's own instructions)
    const double mma1 = bn == 16 ? 41.0 : (bn == 64 ? 50.0 : 66.0);
    // a ring slot is free again one load round trip (about 2.2 us under load) after its MMAs were committed
    const double ring_clk = 4400.0;
    double best_eff = 0.0, best_cost = -1.0;
    for (int tiles_w = tiles_w_min; tiles_w < tiles_w_min + 4; ++tiles_w) {
    const int cw = (s.wo + tiles_w - 1) / tiles_w, wt = cw + s.taps_w - 1;
    if (cw < 8) break;
    for (int r = 1; r <= s.ho && r + s.taps_h - 1 <= 256; ++r) {
        const int nmb = (r * wt + 127) / 128;
        if (nmb > nmb_max) break;
        const size_t px = (size_t)nmb * 128 + (size_t)(s.taps_h - 1) * wt + (s.taps_w - 1);
        const uint32_t sbytes = (uint32_t)(((px * 128) + 1023) / 1024 * 1024);
        // resident weights when they fit beside two patch buffers (one n-tile, no per-class tap masks)
        const bool resident = n_tiles == 1 && !sub_wide && fixed + wall + 2 * (size_t)sbytes <= budget;
        if (!resident && fixed + 4 * bbytes + 2 * (size_t)sbytes > budget) break;
        int nstrips = 2, bstages = 4;
        if (resident) {
            nstrips = (int)((budget - fixed - wall) / sbytes);
            if (nstrips > kSMaxStrips) nstrips = kSMaxStrips;
        } else {
            bstages = (int)((budget - fixed - 2 * (size_t)sbytes) / bbytes);
            if (bstages > kSBStages) bstages = kSBStages;
            if ((long long)bstages > (long long)taps * cchunks) bstages = taps * cchunks;
            nstrips = 2 + (int)((budget - fixed - 2 * (size_t)sbytes - (size_t)bstages * bbytes) / sbytes);
            if (nstrips > kSMaxStrips) nstrips = kSMaxStrips;
        }
        const size_t smem = fixed + (resident ? wall : (size_t)bstages * bbytes) + (size_t)nstrips * sbytes;
        const int tiles_h = (s.ho + r - 1) / r;
        const double eff = (double)s.ho * s.wo / ((double)tiles_h * tiles_w * nmb * 128.0);
        if (eff < 0.70) continue;
        double tap_clk = (double)nmb * 4 * mma1;
        if (!resident && ring_clk / bstages > tap_clk) tap_clk = ring_clk / bstages;
        const double mma_clk = tap_clk * taps * cchunks;
        const double fill_clk = ((double)(r + s.taps_h - 1) * wt * 128.0 + (resident ? 0.0 : (double)taps * bbytes)) *
                                cchunks / 32.0;
        const double tile_clk = (mma_clk > fill_clk ? mma_clk : fill_clk) + 500.0;
        const long long tiles = (long long)s.n * tiles_h * tiles_w * n_tiles;
        // (Tiles of fewer than four M blocks were measured and lose: with two blocks in flight the MMAs of one
        // accumulator wait for each other, 75 clocks per 128 x 64 x 16 MMA instead of 57, and the tile count grows.)
        const double cost = (double)((tiles + sms - 1) / sms) * tile_clk + (resident ? (double)wall / 32.0 : 0.0);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best_eff = eff;
            best.ok = true; best.bn = bn; best.R = r; best.CW = cw; best.Wt = wt; best.nmb = nmb;
            best.strip_bytes = sbytes; best.smem = smem; best.tiles_w = tiles_w;
            best.nstrips = nstrips; best.resident = resident ? 1 : 0; best.bstages = bstages;
            best.nacc = 512 / (bn * nmb) < kSMaxAcc ? 512 / (bn * nmb) : kSMaxAcc;
        }
    }
    }
    if (best_eff < 0.70) best.ok = false;
    return best;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// NHWC bf16 tensor as a 4-D tiled map (c, w, h, n): box = 64 channels x box_w x box_h x 1 image.
bool make_tmap_nhwc_box(CUtensorMap *tm, const void *base, int n, int h, int w, int c, int box_w, int box_h) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return false;
        fn = (EncodeTiledFn)f;
    }
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c * 2, (cuuint64_t)w * c * 2, (cuuint64_t)h * w * c * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


template <int BN>
cudaError_t launch_strip(const CUtensorMap &ta, const CUtensorMap &tw, const StripGemm &g, size_t smem,
                         const float *bias, int *err, cudaStream_t st) {
    static PerDevice attr;
    if (cudaError_t e = max_dynamic_smem_once(umma_strip_conv_kernel<BN>, 226 * 1024, &attr); e != cudaSuccess) return e;
    static PerDevice carve;
    prefer_max_shared_once(umma_strip_conv_kernel<BN>, &carve);
    const long long total = (long long)g.n * g.tiles_h * g.tiles_w * (g.cn / BN);
    const unsigned grid = (unsigned)(total < strip_sm_count() ? total : strip_sm_count());
    return launch_pdl(umma_strip_conv_kernel<BN>, dim3(grid), dim3(kSThreads), smem, st, ta, tw, g, bias, err);
}

}  // namespace

bool umma_strip_eligible(const UmmaConvShape &s) {
    return plan_strip(s).ok;
}

cudaError_t launch_umma_strip_conv(const UmmaConvShape &s, const void *act, const void *wmat, const float *bias,
                                   void *out, cudaStream_t st, const BnFold *fold) {
    const StripPlan pl = plan_strip(s);
    if (!pl.ok) return cudaErrorInvalidValue;
    StripGemm g;
    g.n = s.n; g.ho = s.ho; g.wo = s.wo; g.cn = s.cn; g.ca = s.ca; g.kh = s.taps_h; g.kw = s.taps_w;
    g.lower_h = s.lower_h; g.lower_w = s.lower_w;
    g.R = pl.R; g.CW = pl.CW; g.Wt = pl.Wt; g.rows_in = pl.R + s.taps_h - 1; g.nmb = pl.nmb;
    g.tiles_h = (s.ho + pl.R - 1) / pl.R; g.tiles_w = (s.wo + pl.CW - 1) / pl.CW;
    g.strip_bytes = pl.strip_bytes;
    g.nacc = pl.nacc;
    g.f16 = call_f16();
    g.nstrips = pl.nstrips; g.resident = pl.resident; g.bstages = pl.bstages;
    g.nissue = pl.nmb < kSIssuers ? pl.nmb : kSIssuers;
    g.blockdiag = s.blockdiag;
    g.sub_cin = s.sub_cin; g.sub_hin = s.sub_hin; g.sub_win = s.sub_win;
    g.sub_wide = (s.sub_cin > 0 && s.cn != 16) ? 1 : 0;
    for (int c = 0; c < 4; ++c) g.sub_mask[c] = s.sub_mask[c];
    int cols = pl.nacc * pl.nmb * pl.bn, p2 = 32;
    while (p2 < cols) p2 <<= 1;
    g.tmem_cols = (uint32_t)p2;
    g.out = (__nv_bfloat16 *)out;
    g.fold = fold ? *fold : BnFold{nullptr, nullptr, nullptr, nullptr, nullptr, 0.f, nullptr};
    CUtensorMap ta, tw;
    if (!make_tmap_nhwc_box(&ta, act, s.n, s.ha, s.wa, s.ca, pl.Wt, g.rows_in)) return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tw, wmat, s.cn, (long long)s.taps_h * s.taps_w * (s.blockdiag ? 64 : s.ca), pl.bn, 64))
        return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    if (pl.bn == 16) return launch_strip<16>(ta, tw, g, pl.smem, bias, err, st);
    if (pl.bn == 64) return launch_strip<64>(ta, tw, g, pl.smem, bias, err, st);
    return launch_strip<128>(ta, tw, g, pl.smem, bias, err, st);
}

// ---- stride-2 backward data of a small-C_in layer as a sub-pixel convolution -------------------------
namespace {

// dZ row offsets d = (a + pad - r) / 2 over both parities a and all taps r with a + pad - r even
void subpixel_range(int pad, int k, int *dmin, int *dmax) {
    bool any = false;
    for (int a = 0; a < 2; ++a)
        for (int r = 0; r < k; ++r) {
            const int t = a + pad - r;
            if (t & 1) continue;
            const int d = t / 2;                       // t even: exact
            if (!any || d < *dmin) *dmin = d;
            if (!any || d > *dmax) *dmax = d;
            any = true;
        }
}

__global__ void subpixel_weights_kernel(const __nv_bfloat16 *__restrict__ w, const float *__restrict__ s_vec,
                                        __nv_bfloat16 *__restrict__ wsub, int c_out, int cin, int kh, int kw,
                                        int pad_h, int pad_w, int th, int tw, int dmin_h, int dmin_w, int f16) {
    pdl_wait();
    pdl_launch_dependents();
    const int total = 16 * th * tw * c_out;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int co = idx % c_out;
        int t = idx / c_out;
        const int tq = t % tw; t /= tw;
        const int tr = t % th;
        const int row = t / th, a = row >> 3, e = row & 7, b = e / cin, ci = e - b * cin;
        const int r = a + pad_h - 2 * (dmin_h + tr), q = b + pad_w - 2 * (dmin_w + tq);
        float v = 0.f;
        if (b < 2 && r >= 0 && r < kh && q >= 0 && q < kw)
            v = (s_vec ? s_vec[co] : 1.f) * load_h16(w + (((size_t)co * kh + r) * kw + q) * cin + ci, f16);
        reinterpret_cast<uint16_t *>(wsub)[idx] = pack1_h16(v, f16);
    }
}

}  // namespace

namespace {
__global__ void subpixel_wide_weights_kernel(const __nv_bfloat16 *__restrict__ w, const float *__restrict__ s_vec,
                                             __nv_bfloat16 *__restrict__ wsub, int c_out, int cin, int kh, int kw,
                                             int pad_h, int pad_w, int th, int tw, int dmin_h, int dmin_w, int f16) {
    pdl_wait();
    pdl_launch_dependents();
    const long long total = 4LL * cin * th * tw * c_out;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int co = (int)(idx % c_out);
        long long t = idx / c_out;
        const int tq = (int)(t % tw); t /= tw;
        const int tr = (int)(t % th); t /= th;
        const int ci = (int)(t % cin), cls = (int)(t / cin), a = cls >> 1, b = cls & 1;
        const int r = a + pad_h - 2 * (dmin_h + tr), q = b + pad_w - 2 * (dmin_w + tq);
        float v = 0.f;
        if (r >= 0 && r < kh && q >= 0 && q < kw)
            v = (s_vec ? s_vec[co] : 1.f) * load_h16(w + (((size_t)co * kh + r) * kw + q) * cin + ci, f16);
        reinterpret_cast<uint16_t *>(wsub)[idx] = pack1_h16(v, f16);
    }
}
}  // namespace

bool subpixel_wide_shape(const Problem &pb, UmmaConvShape *s) {
    if (pb.groups != 1 || pb.stride_h != 2 || pb.stride_w != 2 || pb.dil_h != 1 || pb.dil_w != 1) return false;
    if (pb.c_in % 64 || pb.c_out % 64 || pb.c_in > 1024 || pb.kh < 2 || pb.kw < 2 || pb.kh > 8 || pb.kw > 8) return false;
    if (pb.pin >= (1LL << 30) || pb.p >= (1LL << 30)) return false;
    int dmin_h = 0, dmax_h = 0, dmin_w = 0, dmax_w = 0;
    subpixel_range(pb.pad_h, pb.kh, &dmin_h, &dmax_h);
    subpixel_range(pb.pad_w, pb.kw, &dmin_w, &dmax_w);
    const int th = dmax_h - dmin_h + 1, tw = dmax_w - dmin_w + 1;
    if (th * tw > 32) return false;
    *s = UmmaConvShape{pb.n, pb.h_out, pb.w_out, pb.c_out, (pb.h_in + 1) / 2, (pb.w_in + 1) / 2, 4 * pb.c_in,
                       th, tw, dmin_h, dmin_w, 1, 1, 1, 1};
    s->sub_cin = pb.c_in; s->sub_hin = pb.h_in; s->sub_win = pb.w_in;
    for (int cls = 0; cls < 4; ++cls) {
        unsigned m = 0;
        for (int tr = 0; tr < th; ++tr)
            for (int tq = 0; tq < tw; ++tq) {
                const int r = (cls >> 1) + pb.pad_h - 2 * (dmin_h + tr), q = (cls & 1) + pb.pad_w - 2 * (dmin_w + tq);
                if (r >= 0 && r < pb.kh && q >= 0 && q < pb.kw) m |= 1u << (tr * tw + tq);
            }
        if (!m) return false;                          // a class without taps: its outputs are plain zeros
        s->sub_mask[cls] = m;
    }
    return true;
}

bool subpixel_dgrad_shape(const Problem &pb, UmmaConvShape *s) {
    if (pb.groups != 1 || pb.c_in > 4 || pb.stride_h != 2 || pb.stride_w != 2 || pb.dil_h != 1 || pb.dil_w != 1)
        return false;
    if (pb.c_out % 64 || pb.c_out > 1024 || pb.kh > 32 || pb.kw > 32 || pb.pin >= (1LL << 30)) return false;
    int dmin_h = 0, dmax_h = 0, dmin_w = 0, dmax_w = 0;
    subpixel_range(pb.pad_h, pb.kh, &dmin_h, &dmax_h);
    subpixel_range(pb.pad_w, pb.kw, &dmin_w, &dmax_w);
    *s = UmmaConvShape{pb.n, pb.h_out, pb.w_out, pb.c_out, (pb.h_in + 1) / 2, (pb.w_in + 1) / 2, 16,
                       dmax_h - dmin_h + 1, dmax_w - dmin_w + 1, dmin_h, dmin_w, 1, 1, 1, 1};
    s->sub_cin = pb.c_in; s->sub_hin = pb.h_in; s->sub_win = pb.w_in;
    return true;
}

size_t subpixel_weight_bytes(const Problem &pb) {
    UmmaConvShape s;
    if (subpixel_dgrad_shape(pb, &s)) return (size_t)16 * s.taps_h * s.taps_w * pb.c_out * sizeof(__nv_bfloat16);
    if (subpixel_wide_shape(pb, &s)) return (size_t)s.cn * s.taps_h * s.taps_w * pb.c_out * sizeof(__nv_bfloat16);
    return 0;
}

cudaError_t launch_subpixel_weights(const Problem &pb, const void *w, const float *s_vec, void *wsub,
                                    cudaStream_t st) {
    UmmaConvShape s;
    if (!subpixel_dgrad_shape(pb, &s)) {
        if (!subpixel_wide_shape(pb, &s)) return cudaErrorInvalidValue;
        const long long total = (long long)s.cn * s.taps_h * s.taps_w * pb.c_out;
        const long long blocks = (total + 255) / 256;
        return launch_pdl(subpixel_wide_weights_kernel, dim3((unsigned)(blocks < 2368 ? blocks : 2368)), dim3(256), 0, st,
                          (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)wsub, pb.c_out, pb.c_in, pb.kh, pb.kw,
                          pb.pad_h, pb.pad_w, s.taps_h, s.taps_w, s.lower_h, s.lower_w, call_f16());
    }
    const int total = 16 * s.taps_h * s.taps_w * pb.c_out;
    return launch_pdl(subpixel_weights_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st,
                      (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)wsub, pb.c_out, pb.c_in, pb.kh, pb.kw,
                      pb.pad_h, pb.pad_w, s.taps_h, s.taps_w, s.lower_h, s.lower_w, call_f16());
}

}  // namespace convbn
