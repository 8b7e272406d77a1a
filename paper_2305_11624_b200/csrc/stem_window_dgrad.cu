// Backward data of a first-layer ("stem") convolution with stride 2 and very few input channels:
//     dX = omega'_rot (*) dZ     (Sec. 3.2.1; Table 2, Tune row)
// as a SCATTER GEMM.  One dZ row (128 output pixels x C_out channels, one TMA box) is the A operand; the B
// operand is the whole weight tensor as a matrix [(r, q, c)][co] (32 columns per filter row r: kw <= 8 taps x 4
// channel slots, scaled by s[co], resident in shared memory).  One MMA therefore produces, for every filter row
// r at once, the contribution of that dZ row to input row 2 ho + r - pad_h, still in "window" form: accumulator
// element (wo, 4 q + c) belongs to input pixel 2 wo + q - pad_w.  The contraction length is C_out only (no taps
// inside K), N is up to 256: 4 k-steps of a 128 x 224 x 16 MMA per dZ row for a 7 x 7 stem.
//
// Tensor memory holds a ring of 16 blocks of 32 columns, one per input row in flight; the kh blocks a dZ row
// touches are consecutive in the ring, the blocks of rows that no later dZ row reaches are drained: the
// epilogue adds the up to four window positions that meet one input pixel (a shift over accumulator rows,
// done through shared memory), rounds to bf16 and writes the input row with coalesced 16-byte stores.
// A CTA owns a contiguous range of dZ rows and the input rows 2 ho, 2 ho + 1 (padded coordinates) that go with
// them; it also runs the (kh - 1) / 2 dZ rows before its range, whose contributions its first rows need.
//
// Warps: 0 dZ producer (TMA ring), 1 MMA issuer and tensor-memory owner, 2-3 help with set-up, 4-19 four
// epilogue groups that take completed rows in turn.  Every wait is bounded.
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kDgGroups = 4;                 // epilogue groups of four warps
constexpr int kDgThreads = 32 * (4 + 4 * kDgGroups);
constexpr int kDgSlots = 6;                  // dZ rows in the TMA ring (16 KB each)
constexpr int kDgBlocks = 16;                // accumulator blocks of 32 columns

struct WinDgrad {
    int n, h_in, w_in, h_out, w_out, c_out, kh, kw, pad_h, pad_w;
    int halo;                                // (kh - 1) / 2 dZ rows before a segment
    long long total_rows;                    // n * h_out
    const float *s_vec;                      // per-channel scale folded into the weights (NULL: 1)
    int f16;                                 // 16-bit storage type: 0 bf16, 1 IEEE half
};

struct WinDgCtl {
    uint64_t dz_full[kDgSlots], dz_empty[kDgSlots];
    uint64_t blk_full[kDgBlocks], blk_empty[kDgBlocks];
    uint32_t tmem_base;
    int abort_flag;
    unsigned short nrow_of[256];             // weight element (r, q, c) -> row r 32 + 4 q + c of the resident matrix
};

// A segment: the rows [a, b) of image img that this CTA owns; processing starts `halo` rows earlier.
struct DgSegment { int img, a, b, first; };
__device__ __forceinline__ bool dg_next_segment(long long &cur, long long hi, int h_out, int halo, DgSegment &sg) {
    if (cur >= hi) return false;
    const long long img = cur / h_out;
    const int a = (int)(cur - img * h_out);
    long long end = (img + 1) * (long long)h_out;
    if (end > hi) end = hi;
    sg.img = (int)img; sg.a = a; sg.b = (int)(end - img * h_out);
    sg.first = a - halo < 0 ? 0 : a - halo;
    cur = end;
    return true;
}

template <int C>
__global__ void __launch_bounds__(kDgThreads) stem_window_dgrad_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                                      const WinDgrad g,
                                                                      const __nv_bfloat16 *__restrict__ w,
                                                                      __nv_bfloat16 *__restrict__ dx, int *err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *dzs = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);      // kDgSlots x [128 px][128 B]
    uint8_t *wres = dzs + (size_t)kDgSlots * 16384;                                  // [kh * 32 rows][128 B], swizzled
    float *xch = (float *)(wres + (size_t)g.kh * 32 * 128);                           // per group [6 q][4 c][128]
    uint8_t *rowbuf = (uint8_t *)(xch + kDgGroups * 6 * 4 * 128);                     // per group 2048 B
    WinDgCtl *ctl = (WinDgCtl *)(rowbuf + kDgGroups * 2048);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &ctl->abort_flag;
    const long long row_lo = g.total_rows * blockIdx.x / gridDim.x, row_hi = g.total_rows * (blockIdx.x + 1) / gridDim.x;
    const int kh = g.kh;

    if (threadIdx.x == 0) {
        CONVBN_TRACE_POINT(0);
        for (int s = 0; s < kDgSlots; ++s) { mbar_init(&ctl->dz_full[s], 1); mbar_init(&ctl->dz_empty[s], 1); }
        for (int s = 0; s < kDgBlocks; ++s) { mbar_init(&ctl->blk_full[s], 1); mbar_init(&ctl->blk_empty[s], 4); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_dz);
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, 512);
        tmem_relinquish();
    }
    pdl_wait();
    {
        // resident weights: row n = r 32 + 4 q + c, column co: s[co] w[co][r][q][c], zeros in the unused slots
        uint4 *z4 = (uint4 *)wres;
        for (int i = threadIdx.x; i < kh * 32 * 8; i += kDgThreads) z4[i] = make_uint4(0, 0, 0, 0);
        const int rowlen = kh * g.kw * C, total = g.c_out * rowlen;
        if ((int)threadIdx.x < rowlen) {           // the only divisions of the set-up: once per weight-row position
            const int rem = threadIdx.x, c = rem % C, t2 = rem / C, q = t2 % g.kw, r = t2 / g.kw;
            ctl->nrow_of[rem] = (unsigned short)(r * 32 + 4 * q + c);
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        // every accumulator block starts from zero (and is cleared again by whoever drains it), so that all
        // MMAs accumulate and one dZ row needs a single MMA over its kh blocks
        if (warp >= 4 && warp < 8) {
            const uint32_t t0 = ctl->tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
            for (int b = 0; b < kDgBlocks; ++b) tmem_st_32x32_fill(t0 + (uint32_t)b * 32u, 0u);
            tmem_st_wait();
        }
        // 16-byte loads (8 weights), a thread's loads issued together; channel = e / rowlen by a multiply with the
        // rounded-up reciprocal (e < 2^14: the estimate is exact or one too large, fixed up below)
        const uint32_t inv = (65536u + (uint32_t)rowlen - 1u) / (uint32_t)rowlen;
        const uint4 *wsrc = (const uint4 *)w;
        const int n8 = total / 8;                      // C_out = 64: total is a multiple of 8
        for (int base = threadIdx.x; base < n8; base += 2 * kDgThreads) {
            uint4 val[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) val[k] = base + k * kDgThreads < n8 ? __ldg(wsrc + base + k * kDgThreads) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (base + k * kDgThreads >= n8) break;
                const uint32_t wd[4] = {val[k].x, val[k].y, val[k].z, val[k].w};
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    const int e = (base + k * kDgThreads) * 8 + h;
                    int co = (int)(((uint32_t)e * inv) >> 16);
                    int rem = e - co * rowlen;
                    if (rem < 0) { --co; rem += rowlen; }      // the rounded-up reciprocal can overshoot by one
                    const int nrow = ctl->nrow_of[rem];
                    const float wv = unpack_h16((uint16_t)(wd[h >> 1] >> ((h & 1) * 16)), g.f16);
                    const float v = (g.s_vec ? g.s_vec[co] : 1.f) * wv;
                    *(uint16_t *)(wres + (size_t)nrow * 128 + ((((co >> 3) ^ (nrow & 7)) & 7) << 4) + (co & 7) * 2) = pack1_h16(v, g.f16);
                }
            }
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
    const uint32_t tmem_base = ctl->tmem_base;
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(2);

    if (warp == 0) {
        // ---------------- dZ producer ----------------
        if (elect_one()) {
            long long cur = row_lo;
            DgSegment sg;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            while (ok && dg_next_segment(cur, row_hi, g.h_out, g.halo, sg))
                for (int ho = sg.first; ho < sg.b; ++ho) {
                    { CONVBN_TRACE_T0();
                    if (!mbar_wait_bounded(&ctl->dz_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    CONVBN_TRACE_ACC(12); }
                    mbar_arrive_expect_tx(&ctl->dz_full[s], 16384u);
                    tma_load_3d(dzs + (size_t)s * 16384, &tm_dz, &ctl->dz_full[s], 0, 0, sg.img * g.h_out + ho);
                    ++issued;
                    if (++s == kDgSlots) { s = 0; ph ^= 1u; }
                }
            if (!ok) {
                atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1;
                for (int j = issued > kDgSlots ? issued - kDgSlots : 0; j < issued; ++j)
                    mbar_wait_bounded(&ctl->dz_full[j % kDgSlots], (uint32_t)(j / kDgSlots) & 1u, nullptr, 200000000ull);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            const uint32_t hi = smem_desc_hi_sw128(1024);
            const uint32_t dz_lo = smem_desc_lo(smem_u32(dzs), 16), w_lo = smem_desc_lo(smem_u32(wres), 16);
            // blocks [first, first + nb) of the ring (wrapping at 16), filter rows r0 .. r0 + nb - 1
            auto issue = [&](uint32_t a_lo, uint32_t seq_first, int r0, int nb) {
                while (nb > 0) {
                    const uint32_t blk = seq_first % kDgBlocks;
                    int run = (int)(kDgBlocks - blk);
                    if (run > nb) run = nb;
                    const uint32_t idesc = idesc_h16_f32(128, 32 * run, 0, 0, g.f16);
                    const uint32_t d = tmem_base + blk * 32u, b_lo = w_lo + (uint32_t)r0 * 256u;   // 32 rows x 128 B per r
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16_ss_halves<true>(d, a_lo + (uint32_t)k * 2u, hi, b_lo + (uint32_t)k * 2u, hi, idesc);
                    seq_first += (uint32_t)run; r0 += run; nb -= run;
                }
            };
            long long cur = row_lo;
            DgSegment sg;
            int s = 0;
            uint32_t ph = 0, seq = 0;          // seq: input rows allocated so far (block = seq % 16)
            bool ok = true;
            while (ok && dg_next_segment(cur, row_hi, g.h_out, g.halo, sg)) {
                // padded input row 2 ho + r of this segment lives in block (seq_base + 2 (ho - first) + r) % 16
                const uint32_t seq_base = seq;
                for (int ho = sg.first; ho < sg.b && ok; ++ho) {
                    const uint32_t row0 = seq_base + 2u * (uint32_t)(ho - sg.first);
                    const int nnew = ho == sg.first ? kh : (kh < 2 ? kh : 2), nold = kh - nnew;
                    // blocks taken for rows never touched before must have been drained by their last user
                    { CONVBN_TRACE_T0();
                    for (int j = 0; j < nnew && ok; ++j) {
                        const uint32_t sq = row0 + (uint32_t)(nold + j);
                        if (sq >= kDgBlocks && !mbar_spin_bounded(&ctl->blk_empty[sq % kDgBlocks], ((sq / kDgBlocks) & 1u) ^ 1u, abort_flag))
                            ok = false;
                    }
                    CONVBN_TRACE_ACC(13); }
                    if (!ok) break;
                    { CONVBN_TRACE_T0();
                    if (!mbar_spin_bounded(&ctl->dz_full[s], ph, abort_flag)) { ok = false; break; }
                    CONVBN_TRACE_ACC(14); }
                    tc_fence_after_sync();
                    const uint32_t a_lo = dz_lo + (uint32_t)s * (16384u >> 4);
                    issue(a_lo, row0, 0, kh);
                    umma_commit(&ctl->dz_empty[s]);
                    // rows no later dZ row of the segment reaches: 2 ho and 2 ho + 1, everything at the segment's end
                    const int ndone = ho == sg.b - 1 ? kh : (kh < 2 ? kh : 2);
                    for (int j = 0; j < ndone; ++j) umma_commit(&ctl->blk_full[(row0 + (uint32_t)j) % kDgBlocks]);
                    seq = row0 + (uint32_t)ndone;
                    if (++s == kDgSlots) { s = 0; ph ^= 1u; }
                }
            }
            CONVBN_TRACE_POINT(6);
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else if (warp >= 4) {
        // ---------------- epilogue: completed input rows, taken in turn by the two groups ----------------
        const int grp = (warp - 4) >> 2, quarter = warp & 3, j = quarter * 32 + lane, gt = (warp & 3) * 32 + lane;
        float *tile = xch + (size_t)grp * (6 * 4 * 128);
        uint8_t *rbuf = rowbuf + (size_t)grp * 2048;
        const uint32_t bar_id = 2u + (uint32_t)grp;
        long long cur = row_lo;
        DgSegment sg;
        uint32_t seq = 0, done = 0;
        bool ok = true;
        while (ok && dg_next_segment(cur, row_hi, g.h_out, g.halo, sg)) {
            const uint32_t seq_base = seq;
            for (int ho = sg.first; ho < sg.b && ok; ++ho) {
                const uint32_t row0 = seq_base + 2u * (uint32_t)(ho - sg.first);
                const int ndone = ho == sg.b - 1 ? kh : (kh < 2 ? kh : 2);
                for (int jr = 0; jr < ndone && ok; ++jr, ++done) {
                    if ((int)(done % kDgGroups) != grp) continue;
                    const uint32_t sq = row0 + (uint32_t)jr, blk = sq % kDgBlocks;
                    { CONVBN_TRACE_T0();
                    ok = __all_sync(0xffffffffu, mbar_spin_bounded(&ctl->blk_full[blk], (sq / kDgBlocks) & 1u, abort_flag));
                    if (warp == 4 && lane == 0) CONVBN_TRACE_ACC(15); }
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int rp = 2 * ho + jr, rho = rp - g.pad_h;          // padded / real input row
                    const bool stored = rp >= 2 * sg.a && (rp < 2 * sg.b || sg.b == g.h_out) && rho >= 0 && rho < g.h_in;
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + blk * 32u + ((uint32_t)(quarter * 32) << 16);
                    { CONVBN_TRACE_T0();
                    if (stored) {
                        tmem_ld_32x32(taddr, v);
                        tmem_ld_wait();
                    }
                    if (warp == 4 && lane == 0) CONVBN_TRACE_ACC(4); }
                    { CONVBN_TRACE_T0();
                    tmem_st_32x32_fill(taddr, 0u);        // the block's next user accumulates into zeros
                    tmem_st_wait();
                    if (warp == 4 && lane == 0) CONVBN_TRACE_ACC(5); }
                    CONVBN_TRACE_T0();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->blk_empty[blk]);
                    if (!stored) continue;
                    // window positions q >= 2 of this accumulator row belong to pixels that later rows' threads own
#pragma unroll
                    for (int q = 2; q < 8; ++q)
#pragma unroll
                        for (int c = 0; c < C; ++c) tile[((q - 2) * 4 + c) * 128 + j] = __uint_as_float(v[4 * q + c]);
                    named_bar_sync(bar_id, 128);
                    // padded pixel u = 2 j + b gets window position q = b + 2 t of accumulator row j - t, t = 0 .. 3
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const int p = 2 * j + b - g.pad_w;
#pragma unroll
                        for (int c = 0; c < C; ++c) {
                            float acc = __uint_as_float(v[4 * b + c]);
#pragma unroll
                            for (int t = 1; t < 4; ++t)
                                if (j - t >= 0) acc += tile[((b + 2 * t - 2) * 4 + c) * 128 + j - t];
                            if (p >= 0 && p < g.w_in) *(uint16_t *)(rbuf + ((size_t)p * C + c) * 2) = pack1_h16(acc, g.f16);
                        }
                    }
                    named_bar_sync(bar_id, 128);
                    {
                        const int n16 = g.w_in * C * 2 / 16;
                        uint4 *dst = (uint4 *)(dx + ((size_t)sg.img * g.h_in + rho) * g.w_in * C);
                        for (int i = gt; i < n16; i += 128) dst[i] = ((const uint4 *)rbuf)[i];
                    }
                    if (warp == 4 && lane == 0) CONVBN_TRACE_ACC(7);
                }
                seq = row0 + (uint32_t)ndone;
            }
        }
        if (warp == 4 && lane == 0) CONVBN_TRACE_POINT(10);
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(11);
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

// ---- host side --------------------------------------------------------------------------------------
namespace {
size_t dgrad_window_smem(const Problem &pb) {
    return 1024 + (size_t)kDgSlots * 16384 + (size_t)pb.kh * 32 * 128 + kDgGroups * 6 * 4 * 128 * sizeof(float) + kDgGroups * 2048 +
           sizeof(WinDgCtl) + 64;
}

template <int C>
cudaError_t launch_window_dgrad(const CUtensorMap &tdz, const WinDgrad &g, size_t smem, unsigned grid, const void *w,
                                void *dx, int *err, cudaStream_t st) {
    static PerDevice attr, carve;
    if (cudaError_t e = max_dynamic_smem_once(stem_window_dgrad_kernel<C>, 227 * 1024, &attr); e != cudaSuccess) return e;
    prefer_max_shared_once(stem_window_dgrad_kernel<C>, &carve);
    return launch_pdl(stem_window_dgrad_kernel<C>, dim3(grid), dim3(kDgThreads), smem, st, tdz, g,
                      (const __nv_bfloat16 *)w, (__nv_bfloat16 *)dx, err);
}
}  // namespace

bool stem_window_dgrad_eligible(const Problem &pb) {
    if (pb.groups != 1 || pb.c_in > 4 || pb.stride_w != 2 || pb.stride_h != 2 || pb.dil_h != 1 || pb.dil_w != 1) return false;
    if (pb.kw > 8 || pb.kh > 8 || pb.kh < 2 || pb.c_out != 64 || pb.w_in % 8 || pb.w_out > 128) return false;
    if (pb.w_in + pb.pad_w > 256 || pb.pad_h > 64 || pb.pad_w > 64 || (size_t)pb.w_in * pb.c_in * 2 > 2048) return false;
    if (pb.p >= (1LL << 30) || pb.pin >= (1LL << 30)) return false;
    return dgrad_window_smem(pb) <= 226 * 1024;
}

cudaError_t launch_stem_window_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                                     cudaStream_t st) {
    if (!stem_window_dgrad_eligible(pb)) return cudaErrorInvalidValue;
    WinDgrad g;
    g.n = pb.n; g.h_in = pb.h_in; g.w_in = pb.w_in; g.h_out = pb.h_out; g.w_out = pb.w_out; g.c_out = pb.c_out;
    g.kh = pb.kh; g.kw = pb.kw; g.pad_h = pb.pad_h; g.pad_w = pb.pad_w; g.halo = (pb.kh - 1) / 2;
    g.total_rows = (long long)pb.n * pb.h_out; g.s_vec = s_vec; g.f16 = call_f16();
    // input rows below the last one any output row reaches have no gradient: the kernel never visits them
    const int reached = 2 * (pb.h_out - 1) + pb.kh - pb.pad_h;       // first real row that is not reached
    if (reached < pb.h_in) {
        const size_t row_bytes = (size_t)pb.w_in * pb.c_in * 2;
        cudaError_t e = cudaMemset2DAsync((char *)dx + (size_t)reached * row_bytes, (size_t)pb.h_in * row_bytes, 0,
                                          (size_t)(pb.h_in - reached) * row_bytes, (size_t)pb.n, st);
        if (e != cudaSuccess) return e;
    }
    CUtensorMap tdz;
    const unsigned long long dims[3] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                        (unsigned long long)pb.n * pb.h_out};
    const unsigned long long str[3] = {0, (unsigned long long)pb.c_out * 2, (unsigned long long)pb.w_out * pb.c_out * 2};
    const unsigned int box[3] = {64, 128, 1};
    if (!make_tmap_tiled_bf16(&tdz, dz, 3, dims, str, box)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    const long long sms = device_sm_count();
    const unsigned grid = (unsigned)(g.total_rows < sms ? g.total_rows : sms);
    const size_t smem = dgrad_window_smem(pb);
    switch (pb.c_in) {
        case 1: return launch_window_dgrad<1>(tdz, g, smem, grid, w, dx, err, st);
        case 2: return launch_window_dgrad<2>(tdz, g, smem, grid, w, dx, err, st);
        case 3: return launch_window_dgrad<3>(tdz, g, smem, grid, w, dx, err, st);
        default: return launch_window_dgrad<4>(tdz, g, smem, grid, w, dx, err, st);
    }
}

}  // namespace convbn
