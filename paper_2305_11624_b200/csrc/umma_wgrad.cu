// Weight-gradient implicit GEMM on the sm_100a tensor cores:  domega' = dZ (.) X  (Sec. 3.2.1; Table 2,
// Tune row), the reduction over all N H_out W_out output pixels.
//
// GEMM view: D[k][co] = sum_p Xcol[p][k] dZ[p][co] with k = (tap, ci).  Both operands have the
// reduction index p as their slow axis in NHWC memory, so both are fed to tcgen05.mma as MN-major
// tiles: the A tile is two [64 pixels][64 channels] im2col loads of X (two consecutive 64-wide slices
// of k), the B tile is BN/64 plain [64 pixels][64 channels] boxes of dZ.  The pixel range is cut into
// `splits` slices (grid.z); every CTA accumulates its slice in tensor memory in fp32 and writes one
// fp32 partial tile part[split][k][co].  A second kernel adds the slices in fixed order and forms
// domega, dgamma, ... from the fp32 sums (never from rounded values).
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kWM = 128;          // k rows per tile (two 64-channel slices)
constexpr int kWP = 64;           // pixels per stage (reduction depth per stage)
constexpr int kWUmmaK = 16;
constexpr int kWMaxStages = 8;
constexpr int kWThreads = 192;
constexpr uint32_t kChunkBytes = kWP * 64 * 2;   // one [64 pixels][64 channels] bf16 box

struct WgradGemm {
    int ho, wo, c_in, c_out, taps_w;
    int lower_h, lower_w, stride_h, stride_w, dil_h, dil_w;
    int kdim;               // taps * c_in
    long long p;            // output pixels
    long long per_split;    // pixels per slice (multiple of 64)
    int stages;
    int blockdiag;          // grouped conv: c_in = 64 here, k rows are (tap, channel of block blockIdx.y)
    // Small-C_in ("stem") mode: tm_x is the 5-D window view of the packed input (one 64-wide slice per
    // filter row), tm_dz a 4-D map of dZ; a "pixel block" is a 4 x 16 patch of output pixels.
    int stem, stem_tiles_w, stem_tiles_h;
    int no_ones;            // 1: no slice of ones (the packed stem input carries a constant-1 slot instead)
    int f16;                // 16-bit storage type: 0 bf16, 1 IEEE half
};

struct WgradSmemCtl {
    uint64_t full[kWMaxStages];
    uint64_t empty[kWMaxStages];
    uint64_t tmem_full;
    uint32_t tmem_base;
    int abort_flag;
};

template <int BN>
__global__ void __launch_bounds__(kWThreads) umma_wgrad_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                              const __grid_constant__ CUtensorMap tm_dz,
                                                              const WgradGemm g, float *__restrict__ partials,
                                                              float *__restrict__ bsum,
                                                              unsigned int *__restrict__ counters, int ncounters,
                                                              int *err) {
    extern __shared__ uint8_t smem_raw[];
    constexpr uint32_t kABytes = 2 * kChunkBytes, kBBytes = (BN / 64) * kChunkBytes, kStageBytes = kABytes + kBBytes;
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    WgradSmemCtl *ctl = (WgradSmemCtl *)(tiles + (size_t)g.stages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = g.stages;
    const int k0 = blockIdx.x * kWM;                    // first k row of this tile
    const int n0 = blockIdx.y * BN;                     // first output channel
    const long long p0 = (long long)blockIdx.z * g.per_split;
    const long long p1 = p0 + g.per_split < g.p ? p0 + g.per_split : g.p;
    const int num_kb = (int)((p1 - p0 + kWP - 1) / kWP);
    // The list of 64-row slices is the K / 64 real ones followed by one slice of constant ones: its
    // accumulator rows are sum_p dZ[p][co], the per-channel sums needed for dbeta (Table 2), for free.
    const int nch = g.kdim / 64, c_first = k0 / 64;
    const int a_chunks = nch - c_first >= 2 ? 2 : (nch - c_first >= 1 ? 1 : 0);   // slices loaded by TMA
    const int ones_slot = g.no_ones ? -1 : ((c_first == nch) ? 0 : (c_first + 1 == nch ? 1 : -1));
    int b_chunks = (g.c_out - n0) / 64;
    if (b_chunks > BN / 64) b_chunks = BN / 64;
    volatile int *abort_flag = &ctl->abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        mbar_init(&ctl->tmem_full, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, BN);
        tmem_relinquish();
    }
    // the tensor maps are kernel parameters, not data of an earlier kernel: fetch them before the wait
    if (threadIdx.x == 0) { prefetch_tensormap(&tm_x); prefetch_tensormap(&tm_dz); }
    pdl_wait();                 // global memory only after every earlier kernel has finished
    // counters of the epilogue kernel that runs after this one start from zero
    if (counters && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
        for (int i = threadIdx.x; i < ncounters; i += kWThreads) counters[i] = 0u;
    if (ones_slot >= 0) {
        // 1.0 everywhere (invariant under the swizzle); TMA never writes this slice
        const uint32_t one2 = one_h16(g.f16) * 0x10001u;
        const uint4 ones = make_uint4(one2, one2, one2, one2);
        for (int s = 0; s < stages; ++s) {
            uint4 *dst = (uint4 *)(tiles + (size_t)s * kStageBytes + (size_t)ones_slot * kChunkBytes);
            for (int i = threadIdx.x; i < (int)(kChunkBytes / 16); i += kWThreads) dst[i] = ones;
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // The whole warp runs the loop; lanes 0-1 load the two X slices, lanes 2.. the dZ boxes.
        const uint32_t tx_bytes = (uint32_t)(a_chunks + b_chunks) * kChunkBytes;
        // this lane's X slice: k = tap * c_in + ci is fixed for the whole CTA
        const int kk = k0 + (lane & 1) * 64;
        const int tap = kk / g.c_in, ci0 = kk - tap * g.c_in + (g.blockdiag ? n0 : 0);
        const int tr = tap / g.taps_w, tq = tap - tr * g.taps_w;
        const uint16_t off_w = (uint16_t)(tq * g.dil_w), off_h = (uint16_t)(tr * g.dil_h);
        int issued = 0, s = 0;
        uint32_t ph = 0;
        bool ok = true;
        // pixel coordinates of the slice start, advanced by 64 pixels per stage without divisions
        uint32_t pp = (uint32_t)p0;
        uint32_t t0 = pp / (uint32_t)g.wo;
        int wo0 = (int)(pp - t0 * (uint32_t)g.wo);
        uint32_t img = t0 / (uint32_t)g.ho;
        int ho0 = (int)(t0 - img * (uint32_t)g.ho);
        for (int kb = 0; kb < num_kb; ++kb) {
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag));
            if (!ok) break;
            const int base_w = g.lower_w + wo0 * g.stride_w, base_h = g.lower_h + ho0 * g.stride_h;
            uint8_t *a_dst = tiles + (size_t)s * kStageBytes, *b_dst = a_dst + kABytes;
            if (lane == 0) mbar_arrive_expect_tx(&ctl->full[s], tx_bytes);
            if (g.stem) {
                // pixel block -> (image, patch row, patch column) of 4 x 16 output pixels
                const uint32_t blk = (uint32_t)(p0 / kWP) + (uint32_t)kb;
                const uint32_t t1 = blk / (uint32_t)g.stem_tiles_w;
                const int pw = (int)(blk - t1 * (uint32_t)g.stem_tiles_w) * 16;
                const uint32_t im = t1 / (uint32_t)g.stem_tiles_h;
                const int phh = (int)(t1 - im * (uint32_t)g.stem_tiles_h) * 4;
                if (lane < a_chunks)
                    tma_load_5d(a_dst + lane * kChunkBytes, &tm_x, &ctl->full[s], 0, pw, phh, c_first + lane, (int)im);
                else if (lane >= 2 && lane - 2 < b_chunks)
                    tma_load_4d(b_dst + (lane - 2) * kChunkBytes, &tm_dz, &ctl->full[s], n0 + (lane - 2) * 64, pw, phh,
                                (int)im);
            } else
            if (lane < a_chunks)
                tma_load_im2col_4d(a_dst + lane * kChunkBytes, &tm_x, &ctl->full[s], ci0, base_w, base_h, (int)img,
                                   off_w, off_h);
            else if (lane >= 2 && lane - 2 < b_chunks)
                tma_load_2d(b_dst + (lane - 2) * kChunkBytes, &tm_dz, &ctl->full[s], n0 + (lane - 2) * 64, (int)pp);
            ++issued;
            if (++s == stages) { s = 0; ph ^= 1u; }
            pp += kWP;
            wo0 += kWP;
            while (wo0 >= g.wo) { wo0 -= g.wo; if (++ho0 == g.ho) { ho0 = 0; ++img; } }
        }
        if (!ok && lane == 0) {
            atomicOr(err, ERRW_TIMEOUT);
            ctl->abort_flag = 1;
            const int first = issued > stages ? issued - stages : 0;
            for (int kb = first; kb < issued; ++kb)
                mbar_wait_bounded(&ctl->full[kb % stages], (uint32_t)(kb / stages) & 1u, nullptr, 200000000ull);
        }
    } else if (warp == 1) {
        if (elect_one()) {
            const uint32_t idesc = idesc_h16_f32(kWM, BN, 1, 1, g.f16);   // both operands MN-major
            const uint32_t hi = smem_desc_hi_sw128(1024);
            const uint32_t tiles_lo = smem_desc_lo(smem_u32(tiles), kChunkBytes);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) {
                    atomicOr(err, ERRW_TIMEOUT);
                    ctl->abort_flag = 1;
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                // 16 pixels = two groups of 8 rows (1024 B apart); 64-channel slices 8192 B apart; descriptors as
                // halves, only the start-address field (16-byte units) moves
                const uint32_t a_lo = tiles_lo + (uint32_t)s * (kStageBytes >> 4), b_lo = a_lo + (kABytes >> 4);
                if (kb == 0) umma_bf16_ss_halves<false>(tmem_base, a_lo, hi, b_lo, hi, idesc);
                else umma_bf16_ss_halves<true>(tmem_base, a_lo, hi, b_lo, hi, idesc);
#pragma unroll
                for (int k = 1; k < kWP / kWUmmaK; ++k)
                    umma_bf16_ss_halves<true>(tmem_base, a_lo + (uint32_t)k * (kWUmmaK * 128 >> 4), hi,
                                              b_lo + (uint32_t)k * (kWUmmaK * 128 >> 4), hi, idesc);
                umma_commit(&ctl->empty[s]);
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(&ctl->tmem_full);
        }
    } else {
        const int quarter = warp & 3;
        const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->tmem_full, 0, abort_flag));
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        if (ok) {
            tc_fence_after_sync();
            const int k = k0 + quarter * 32 + lane;
            const bool row_ok = k < g.kdim;
            const bool sum_row = !g.no_ones && (k == g.kdim);   // first row of the ones slice
            float *brow = bsum + (size_t)blockIdx.z * g.c_out + n0;
            float *orow = g.blockdiag
                              ? partials + (((size_t)blockIdx.z * gridDim.y + blockIdx.y) * g.kdim + (row_ok ? k : 0)) * 64
                              : partials + ((size_t)blockIdx.z * g.kdim + (row_ok ? k : 0)) * g.c_out + n0;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= g.c_out) break;
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *(uint4 *)(orow + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                } else if (sum_row) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *(uint4 *)(brow + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, BN);
}

bool grouped_bd_eligible(const Problem &pb) {
    if (pb.groups <= 1 || pb.cg != pb.cog || pb.cg < 2 || 64 % pb.cg || pb.c_in % 64) return false;
    if (pb.pad_h > 128 || pb.pad_w > 128) return false;
    if ((pb.kh - 1) * pb.dil_h > 255 || (pb.kw - 1) * pb.dil_w > 255) return false;
    if (pb.stride_h > 8 || pb.stride_w > 8) return false;
    if (pb.p >= (1LL << 31) - 256 || pb.pin >= (1LL << 31) - 256) return false;
    return true;
}

bool umma_wgrad_eligible(const Problem &pb) {
    if (pb.groups != 1 || pb.c_in % 64 || pb.c_out % 64) return false;
    if (pb.pad_h > 128 || pb.pad_w > 128) return false;
    if ((pb.kh - 1) * pb.dil_h > 255 || (pb.kw - 1) * pb.dil_w > 255) return false;
    if (pb.stride_h > 8 || pb.stride_w > 8) return false;
    if (pb.p >= (1LL << 31)) return false;
    return true;
}

static int wgrad_bn(const Problem &pb) { return pb.c_out >= 256 ? 256 : (pb.c_out >= 128 ? 128 : 64); }

UmmaWgradPlan umma_wgrad_plan(const Problem &pb) {
    UmmaWgradPlan pl;
    const bool bd = pb.groups > 1;
    const int bn = bd ? 64 : wgrad_bn(pb);
    const long long kd = bd ? (long long)pb.kh * pb.kw * 64 : pb.kdim;
    const long long m_tiles = (kd / 64 + 1 + 1) / 2, n_tiles = (pb.c_out + bn - 1) / bn;   // + the ones slice
    // Resident CTAs: the 64- and 128-wide tiles run two CTAs per SM (their stage rings are sized for it,
    // launch_w), which measured 25-40 % faster than one CTA with a deeper ring; 256-wide tiles own an SM.
    // The slice count minimises  rounds over the resident slots x (pixels per slice + a fixed cost per
    // CTA, in pixels) + a small cost per slice for the epilogue that adds the slices up; a grid a few
    // CTAs larger than the slots would otherwise run a second, nearly empty round.
    const long long slots = (long long)device_sm_count() * (bn == 256 ? 1 : 2), tiles = m_tiles * n_tiles;
    const long long max_splits = (pb.p + 4 * kWP - 1) / (4 * kWP);     // at least 256 pixels per slice
    long long splits = 1;
    double best_cost = -1.0;
    for (long long sp = 1; sp <= max_splits; ++sp) {
        const long long rounds = (tiles * sp + slots - 1) / slots;
        const double cost = (double)rounds * ((double)pb.p / (double)sp + 384.0) + 4.0 * (double)sp;
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; splits = sp; }
        if (tiles * sp > 4 * slots) break;
    }
    long long per = (pb.p + splits - 1) / splits;
    per = (per + kWP - 1) / kWP * kWP;
    pl.per_split = per;
    pl.splits = (int)((pb.p + per - 1) / per);
    wgrad_epilogue_shape(pb, &pl);
    return pl;
}

// k rows per epilogue block (the block's other lanes split the slices): very many slices -> 2 rows x 16
// lanes; few slices or very many blocks -> 32 rows x 1 lane (every block pays a fence and an atomic)
void wgrad_epilogue_shape(const Problem &pb, UmmaWgradPlan *pl) {
    const long long blocks8 = (long long)(pb.c_out / 32) * ((pb.kdim + 7) / 8);
    pl->kr = pl->splits > 192 ? 2 : ((pl->splits <= 8 || blocks8 > 600) && blocks8 / 4 >= device_sm_count() ? 32 : 8);
    // very large weight matrices in few slices: 8 groups of 8 rows per block halve the blocks (and their fences) again
    if (pl->kr == 32 && pl->splits <= 4 && blocks8 / 8 >= 2 * device_sm_count()) pl->kr = 64;
    pl->kt = (pb.kdim + pl->kr - 1) / pl->kr;   // epilogue blocks along k = rows of dotpart
}

template <int BN>
static cudaError_t launch_w(const CUtensorMap &tx, const CUtensorMap &tdz, WgradGemm g, const UmmaWgradPlan &pl,
                            const Problem &pb, float *partials, float *bsum, unsigned int *counters, int *err,
                            cudaStream_t st) {
    constexpr size_t stage = 2 * kChunkBytes + (BN / 64) * kChunkBytes;
    int stages = BN == 128 ? 3 : 4;                    // 128-wide: 3 x 32 KB, so that two CTAs share an SM
    const long long max_kb = (pl.per_split + kWP - 1) / kWP;
    if (stages > max_kb) stages = (int)max_kb;
    g.stages = stages;
    size_t smem = stages * stage + 1024 + sizeof(WgradSmemCtl);
    const size_t floor_smem = (size_t)(228 * 1024) / (512 / BN + 1) + 1024;
    if (smem < floor_smem) smem = floor_smem;
    static PerDevice attr_done;
    if (cudaError_t e = max_dynamic_smem_once(umma_wgrad_kernel<BN>, 210 * 1024, &attr_done); e != cudaSuccess) return e;
    static PerDevice carve;
    prefer_max_shared_once(umma_wgrad_kernel<BN>, &carve);
    dim3 grid((unsigned)((g.kdim / 64 + (g.no_ones ? 1 : 2)) / 2), (unsigned)((pb.c_out + BN - 1) / BN),
              (unsigned)pl.splits);
    return launch_pdl(umma_wgrad_kernel<BN>, grid, dim3(kWThreads), smem, st, tx, tdz, g, partials, bsum, counters,
                      pb.c_out / 32, err);
}

cudaError_t launch_umma_wgrad(const Problem &pb, const UmmaWgradPlan &pl, const void *dz, const void *x,
                              float *partials, float *bsum, unsigned int *counters, cudaStream_t st) {
    WgradGemm g;
    g.ho = pb.h_out; g.wo = pb.w_out; g.c_in = pb.c_in; g.c_out = pb.c_out; g.taps_w = pb.kw;
    g.lower_h = -pb.pad_h; g.lower_w = -pb.pad_w; g.stride_h = pb.stride_h; g.stride_w = pb.stride_w;
    g.dil_h = pb.dil_h; g.dil_w = pb.dil_w; g.kdim = pb.kdim; g.p = pb.p; g.per_split = pl.per_split; g.stages = 1;
    g.blockdiag = pb.groups > 1 ? 1 : 0;
    g.stem = 0; g.stem_tiles_w = g.stem_tiles_h = 1; g.no_ones = 0; g.f16 = call_f16();
    if (g.blockdiag) { g.c_in = 64; g.kdim = pb.kh * pb.kw * 64; }
    const int upper_h = g.lower_h + (pb.h_out - 1) * pb.stride_h - (pb.h_in - 1);
    const int upper_w = g.lower_w + (pb.w_out - 1) * pb.stride_w - (pb.w_in - 1);
    CUtensorMap tx, tdz;
    if (!make_tmap_im2col_bf16(&tx, x, pb.n, pb.h_in, pb.w_in, pb.c_in, g.lower_h, g.lower_w, upper_h, upper_w,
                               pb.stride_h, pb.stride_w, kWP, 64))
        return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tdz, dz, pb.p, pb.c_out, kWP, 64)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    const int bn = g.blockdiag ? 64 : wgrad_bn(pb);
    if (bn == 64) return launch_w<64>(tx, tdz, g, pl, pb, partials, bsum, counters, err, st);
    if (bn == 128) return launch_w<128>(tx, tdz, g, pl, pb, partials, bsum, counters, err, st);
    return launch_w<256>(tx, tdz, g, pl, pb, partials, bsum, counters, err, st);
}

// ---- epilogue over k-major partials ------------------------------------------------------------
// One kernel finishes every parameter gradient (Table 2, Tune row) from the fp32 partial tiles:
//   block (bx, by): 32 output channels x KR k rows x SL lanes over the pixel slices (KR SL = 32,
//   up to 1024 threads), REP such row groups one after the other: (8, 4) when there are few slices, (2, 16)
//   when there are many, (8, 1) x 4 with 256 threads when there are few slices and thousands of blocks
//     acc[k][co] = sum_split part[split][k][co]        (each lane a strided subset, lanes added in order)
//     dw[co][k]  = s[co] acc                           (transposed through shared memory)
//     dotpart[by][co] = sum over the block's k rows of acc * w[co][k]
//   the LAST block to finish for a group of 32 channels (a counter per group, zeroed by the GEMM
//   kernel) adds dotpart over all k blocks and bsum over all slices, lanes strided + a fixed shuffle
//   tree, so the result does not depend on which block came last:
//     dbeta = sum dZ,  db = s dbeta,  dgamma = r (sum_k domega' omega + dbeta (b - mu_hat))
//   plain mode (vec3 == NULL): dw = acc, db = sum dZ if requested.
template <int KR, int SL, int REP>
__global__ void __launch_bounds__(32 * KR * SL, SL == 16 ? 2 : (KR * SL == 8 ? 4 : 1)) wgrad_epilogue_fused_kernel(
    int c_out, int kdim, const float *__restrict__ part, int splits, const float *__restrict__ bsum, int bsplits,
    const __nv_bfloat16 *__restrict__ w, const float *__restrict__ vec3, const float *__restrict__ b,
    const float *__restrict__ mean, float *__restrict__ dw, float *__restrict__ dotpart,
    unsigned int *__restrict__ counters, float *__restrict__ db, float *__restrict__ dgamma,
    float *__restrict__ dbeta, int need_sums, int f16) {
    static_assert(KR * SL <= 32, "at most 32 warps per block");
    // loads in flight per thread: the (2, 16) shape has the most blocks and is held to 32 registers, so
    // that two of its 1024-thread blocks share an SM
    constexpr int NB = SL == 16 ? 4 : 8;
    __shared__ float tile[REP][SL][KR][33];
    __shared__ int is_last;
    pdl_wait();
    pdl_launch_dependents();
    const int tx = threadIdx.x & 31, ty = (threadIdx.x >> 5) % KR, tz = (threadIdx.x >> 5) / KR;
    const int co0 = blockIdx.x * 32, k0 = blockIdx.y * (KR * REP);   // REP groups of KR rows per block
    const size_t slice = (size_t)kdim * c_out;
    // the weights the second phase multiplies with are requested now, together with the partials
    float wv[REP];
#pragma unroll
    for (int rep = 0; rep < REP; ++rep) {
        const int k = k0 + rep * KR + (int)(threadIdx.x % KR), co = co0 + (int)(threadIdx.x / KR);
        wv[rep] = (vec3 && threadIdx.x < 32 * KR && k < kdim) ? load_h16(w + (size_t)co * kdim + k, f16) : 0.f;
    }
    constexpr int NBF = REP > 1 ? 32 / REP : 1;      // slices the preloading path below can take
    if (SL == 1 && REP > 1 && splits <= NBF) {
        // few slices, several row groups: request every value of every group before the first use, so that
        // REP x splits loads are in flight per thread instead of `splits`; same order of additions as below
        float a[REP][NBF];
#pragma unroll
        for (int rep = 0; rep < REP; ++rep) {
            const int k = k0 + rep * KR + ty;
            const float *src = part + (size_t)k * c_out + co0 + tx;
#pragma unroll
            for (int u = 0; u < NBF; ++u) a[rep][u] = (k < kdim && u < splits) ? __ldcg(src + (size_t)u * slice) : 0.f;
        }
#pragma unroll
        for (int rep = 0; rep < REP; ++rep) {
            float tot = 0.f;
#pragma unroll
            for (int u = 0; u < NBF; ++u) tot += a[rep][u];
            tile[rep][tz][ty][tx] = tot;
        }
    } else
#pragma unroll
    for (int rep = 0; rep < REP; ++rep) {
        const int k = k0 + rep * KR + ty;
        // NB independent sums per thread keep NB loads in flight; they are added in a fixed order
        float a[NB];
#pragma unroll
        for (int u = 0; u < NB; ++u) a[u] = 0.f;
        if (k < kdim) {
            const float *src = part + (size_t)k * c_out + co0 + tx;
            int sp = tz;
            for (; sp + (NB - 1) * SL < splits; sp += NB * SL) {
#pragma unroll
                for (int u = 0; u < NB; ++u) a[u] += __ldcg(src + (size_t)(sp + u * SL) * slice);
            }
#pragma unroll
            for (int u = 0; u < NB; ++u)
                if (sp + u * SL < splits) a[u] += __ldcg(src + (size_t)(sp + u * SL) * slice);
        }
        float tot = 0.f;
#pragma unroll
        for (int u = 0; u < NB; ++u) tot += a[u];
        tile[rep][tz][ty][tx] = tot;
    }
    __syncthreads();
    if (threadIdx.x < 32 * KR) {
        const int kk = threadIdx.x % KR, cl = threadIdx.x / KR, co = co0 + cl;
        float d = 0.f;
#pragma unroll
        for (int rep = 0; rep < REP; ++rep) {
            const int k = k0 + rep * KR + kk;
            if (k < kdim) {
                float v = 0.f;
#pragma unroll
                for (int z = 0; z < SL; ++z) v += tile[rep][z][kk][cl];
                const size_t o = (size_t)co * kdim + k;
                dw[o] = (vec3 ? vec3[co] : 1.f) * v;
                d = fmaf(v, wv[rep], d);
            }
        }
        if (vec3) {
#pragma unroll
            for (int o = 1; o < KR; o <<= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (kk == 0) dotpart[(size_t)blockIdx.y * c_out + co] = d;
        }
    }
    if (!need_sums) return;
    // ---- last block of this channel group finishes the per-channel quantities ----
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();        // after the barrier: orders the whole block's dw / dotpart writes before the count
        const unsigned int done = atomicAdd(&counters[blockIdx.x], 1u);
        is_last = (done == gridDim.y - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // Thread (channel ch, row group grp) adds rows grp, grp + ngrp, ... of the dZ sums and of the dot
    // partials: a row's 32 channels are one 128-byte read, a thread's (up to NB) rows are requested
    // together, and the groups are then added in order: one memory round trip instead of one per row.
    {
        __shared__ float fin[2][32][33];
        const int ch = tx, grp = (int)(threadIdx.x >> 5), ngrp = KR * SL;
        float ds = 0.f, dt = 0.f;
        for (int base = grp; base < bsplits; base += ngrp * NB) {
            float v[NB];
#pragma unroll
            for (int u = 0; u < NB; ++u) {
                const int sp = base + u * ngrp;
                v[u] = sp < bsplits ? __ldcg(bsum + (size_t)sp * c_out + co0 + ch) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < NB; ++u) ds += v[u];
        }
        if (vec3)
            for (int base = grp; base < (int)gridDim.y; base += ngrp * NB) {
                float v[NB];
#pragma unroll
                for (int u = 0; u < NB; ++u) {
                    const int t = base + u * ngrp;
                    v[u] = t < (int)gridDim.y ? __ldcg(dotpart + (size_t)t * c_out + co0 + ch) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < NB; ++u) dt += v[u];
            }
        fin[0][grp][ch] = ds;
        fin[1][grp][ch] = dt;
        __syncthreads();
        if (threadIdx.x < 32) {
            const int co = co0 + ch;
            float dsum = 0.f, dot = 0.f;
            for (int gq = 0; gq < ngrp; ++gq) { dsum += fin[0][gq][ch]; dot += fin[1][gq][ch]; }
            if (!vec3) {
                if (db) db[co] = dsum;
            } else {
                const float s = vec3[co], r = vec3[2 * c_out + co];
                dbeta[co] = dsum;
                if (db) db[co] = s * dsum;
                dgamma[co] = r * (dot + dsum * ((b ? b[co] : 0.f) - mean[co]));
            }
        }
    }
    if (threadIdx.x == 0) counters[blockIdx.x] = 0;   // leave the counter clean for the next call
}

cudaError_t launch_wgrad_epilogue_fused(const Problem &pb, const UmmaWgradPlan &pl, const float *partials,
                                        const float *bsum, const void *w, const float *vec3, const float *b,
                                        const float *mean, float *dw, float *dotpart, unsigned int *counters,
                                        float *db, float *dgamma, float *dbeta, bool need_sums, cudaStream_t st) {
    const dim3 grid(pb.c_out / 32, pl.kt);
    const int ns = need_sums ? 1 : 0;
    static PerDevice carve_a, carve_b;
    prefer_max_shared_once(wgrad_epilogue_fused_kernel<8, 4, 1>, &carve_a);
    prefer_max_shared_once(wgrad_epilogue_fused_kernel<2, 16, 1>, &carve_b);
    if (pl.kr == 64)
        return launch_pdl(wgrad_epilogue_fused_kernel<8, 1, 8>, grid, dim3(256), 0, st, pb.c_out, pb.kdim, partials,
                          pl.splits, bsum, pl.splits, (const __nv_bfloat16 *)w, vec3, b, mean, dw, dotpart, counters, db,
                          dgamma, dbeta, ns, call_f16());
    if (pl.kr == 32)                                  // 4 groups of 8 rows, 256 threads: several blocks per SM
        return launch_pdl(wgrad_epilogue_fused_kernel<8, 1, 4>, grid, dim3(256), 0, st, pb.c_out, pb.kdim, partials,
                          pl.splits, bsum, pl.splits, (const __nv_bfloat16 *)w, vec3, b, mean, dw, dotpart, counters, db,
                          dgamma, dbeta, ns, call_f16());
    if (pl.kr == 8)
        return launch_pdl(wgrad_epilogue_fused_kernel<8, 4, 1>, grid, dim3(1024), 0, st, pb.c_out, pb.kdim, partials,
                          pl.splits, bsum, pl.splits, (const __nv_bfloat16 *)w, vec3, b, mean, dw, dotpart, counters, db,
                          dgamma, dbeta, ns, call_f16());
    return launch_pdl(wgrad_epilogue_fused_kernel<2, 16, 1>, grid, dim3(1024), 0, st, pb.c_out, pb.kdim, partials,
                      pl.splits, bsum, pl.splits, (const __nv_bfloat16 *)w, vec3, b, mean, dw, dotpart, counters, db,
                      dgamma, dbeta, ns, call_f16());
}

// ---- small-C_in ("stem") layers -------------------------------------------------------------------
UmmaWgradPlan stem_wgrad_plan(const Problem &pb) {
    UmmaWgradPlan pl;
    const int bn = wgrad_bn(pb);
    const long long patches = (long long)pb.n * ((pb.h_out + 3) / 4) * ((pb.w_out + 15) / 16);
    const long long m_tiles = (stem_krows(pb) + (stem_ones_in_pack(pb) ? 1 : 2)) / 2, n_tiles = (pb.c_out + bn - 1) / bn;
    long long splits = (device_sm_count() + m_tiles * n_tiles - 1) / (m_tiles * n_tiles);
    if (splits > (patches + 3) / 4) splits = (patches + 3) / 4;
    if (splits < 1) splits = 1;
    const long long per = (patches + splits - 1) / splits;
    pl.per_split = per * kWP;                       // in pixels of 4 x 16 patches
    pl.splits = (int)((patches + per - 1) / per);
    pl.kr = 8; pl.kt = 1;
    return pl;
}

// partials: [splits][krows * 64][C_out]; bsum: [splits][C_out]
cudaError_t launch_stem_wgrad(const Problem &pb, const UmmaWgradPlan &pl, const void *dz, const void *x_packed,
                              float *partials, float *bsum, cudaStream_t st) {
    const int krows = stem_krows(pb);
    WgradGemm g;
    g.ho = pb.h_out; g.wo = pb.w_out; g.c_in = 64; g.c_out = pb.c_out; g.taps_w = 1;
    g.lower_h = g.lower_w = 0; g.stride_h = g.stride_w = g.dil_h = g.dil_w = 1;
    g.kdim = krows * 64;
    g.stem = 1; g.stem_tiles_w = (pb.w_out + 15) / 16; g.stem_tiles_h = (pb.h_out + 3) / 4;
    g.no_ones = stem_ones_in_pack(pb) ? 1 : 0;
    g.f16 = call_f16();
    g.p = (long long)pb.n * g.stem_tiles_h * g.stem_tiles_w * kWP;
    g.per_split = pl.per_split; g.stages = 1; g.blockdiag = 0;
    CUtensorMap tx, tdz;
    {
        const unsigned long long dims[5] = {64, (unsigned long long)pb.w_out, (unsigned long long)pb.h_out,
                                            (unsigned long long)krows, (unsigned long long)pb.n};
        unsigned long long str[5];
        stem_window_strides(pb, str);
        const unsigned int box[5] = {64, 16, 4, 1, 1};
        if (!make_tmap_tiled_bf16(&tx, x_packed, 5, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const unsigned long long dims[4] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                            (unsigned long long)pb.h_out, (unsigned long long)pb.n};
        const unsigned long long str[4] = {0, (unsigned long long)pb.c_out * 2,
                                           (unsigned long long)pb.w_out * pb.c_out * 2,
                                           (unsigned long long)pb.h_out * pb.w_out * pb.c_out * 2};
        const unsigned int box[4] = {64, 16, 4, 1};
        if (!make_tmap_tiled_bf16(&tdz, dz, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    Problem q = pb;
    q.kdim = g.kdim;                                   // grid: (kh + 2) / 2 row tiles
    const int bn = wgrad_bn(pb);
    if (bn == 64) return launch_w<64>(tx, tdz, g, pl, q, partials, bsum, nullptr, err, st);
    if (bn == 128) return launch_w<128>(tx, tdz, g, pl, q, partials, bsum, nullptr, err, st);
    return launch_w<256>(tx, tdz, g, pl, q, partials, bsum, nullptr, err, st);
}

// One block per output channel: gathers the kh x kw x C_in real entries out of the krows x 64 padded rows,
// adds the slices in order and finishes domega, db, dgamma, dbeta (Table 2, Tune row) or the plain sums.
__global__ void __launch_bounds__(256) wgrad_epilogue_stem_kernel(int c_out, int kh, int kw, int c_in, int krows, int s2d,
                                                                 int sum_row,
                                                                 const float *__restrict__ part, int splits,
                                                                 const float *__restrict__ bsum,
                                                                 const __nv_bfloat16 *__restrict__ w,
                                                                 const float *__restrict__ vec3,
                                                                 const float *__restrict__ b,
                                                                 const float *__restrict__ mean,
                                                                 float *__restrict__ dw, float *__restrict__ db,
                                                                 float *__restrict__ dgamma,
                                                                 float *__restrict__ dbeta, int need_sums, int f16) {
    __shared__ float red[256];
    const int co = blockIdx.x, kdim = kh * kw * c_in;
    const size_t slice = (size_t)krows * 64 * c_out;
    const float s = vec3 ? vec3[co] : 1.f;
    float dot = 0.f;
    for (int k = threadIdx.x; k < kdim; k += blockDim.x) {
        const int c = k % c_in, t = k / c_in, q = t % kw, r = t / kw;
        const size_t o = (s2d ? (size_t)(r >> 1) * 64 + (q >> 1) * 16 + (r & 1) * 8 + (q & 1) * 4 + c
                              : (size_t)r * 64 + q * 8 + c) * c_out + co;
        float acc = 0.f;
        for (int sp = 0; sp < splits; ++sp) acc += part[(size_t)sp * slice + o];
        dw[(size_t)co * kdim + k] = s * acc;
        if (vec3) dot = fmaf(acc, load_h16(w + (size_t)co * kdim + k, f16), dot);
    }
    float bs = 0.f;
    if (need_sums)
        for (int sp = threadIdx.x; sp < splits; sp += blockDim.x)   // sum dZ: its own array, or k row `sum_row`
            bs += sum_row >= 0 ? part[(size_t)sp * slice + (size_t)sum_row * c_out + co] : bsum[(size_t)sp * c_out + co];
    red[threadIdx.x] = dot;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    const float dot_all = red[0];
    __syncthreads();
    red[threadIdx.x] = bs;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    if (threadIdx.x == 0 && need_sums) {
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

cudaError_t launch_wgrad_epilogue_stem(const Problem &pb, const UmmaWgradPlan &pl, const float *partials,
                                       const float *bsum, const void *w, const float *vec3, const float *b,
                                       const float *mean, float *dw, float *db, float *dgamma, float *dbeta,
                                       bool need_sums, cudaStream_t st) {
    wgrad_epilogue_stem_kernel<<<pb.c_out, 256, 0, st>>>(pb.c_out, pb.kh, pb.kw, pb.c_in, stem_krows(pb), stem_s2d(pb) ? 1 : 0,
                                                         stem_ones_in_pack(pb) ? 3 : -1, partials, pl.splits, bsum,
                                                         (const __nv_bfloat16 *)w, vec3, b, mean, dw, db, dgamma, dbeta,
                                                         need_sums ? 1 : 0, call_f16());
    return cudaGetLastError();
}

}  // namespace convbn
