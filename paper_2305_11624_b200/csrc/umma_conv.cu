// Implicit-GEMM convolution on the sm_100a tensor cores (tcgen05.mma, accumulator in tensor memory),
// operands staged by TMA: the activation operand by im2col-mode loads straight from the NHWC tensor,
// the weight operand by tiled loads of a [C_n][taps * C_a] matrix.  One kernel serves
//   forward        Z  = omega' (*) X + b'      (Sec. 3.1 / 3.3): activation X,  weights omega'
//   backward data  dX = omega'_rot (*) dZ      (Sec. 3.2.1)    : activation dZ, weights omega' with
//                  taps flipped and channel roles swapped (stride-1 convolutions)
// GEMM view (Sec. 3.2.2): M = output pixels, N = output channels, K = taps x input channels.
//
// CTA = 6 warps: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the MMAs, warps 2-5
// move the 128 x BN fp32 accumulator from tensor memory to registers, add the bias, round to bf16
// and store.  A ring of `stages` shared-memory slots decouples loads from MMAs.  Every wait is
// bounded; a wait that gives up sets the device error word and the CTA drains and exits.
#include <mutex>

#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kBM = 128;       // output pixels per tile (UMMA M)
constexpr int kBK = 64;        // K elements per stage = one 128-byte swizzle row of bf16
constexpr int kUmmaK = 16;     // K per tcgen05.mma of kind::f16
constexpr int kMaxStages = 12;
constexpr int kConvThreads = 320;                             // TMA warp, MMA warp, 2 x 4 epilogue warps
constexpr uint32_t kStagingWarpBytes = 32 * 128;              // [32 rows][64 bf16]
constexpr uint32_t kStagingBytes = 8 * kStagingWarpBytes;     // one buffer per epilogue warp

struct ConvGemm {
    int ho, wo;              // output spatial extent
    int cn;                  // output channels (GEMM N)
    int ca;                  // activation channels (multiple of 64)
    int taps_h, taps_w;
    int lower_h, lower_w;    // input coordinate read by output (0,0) at tap (0,0)
    int stride_h, stride_w, dil_h, dil_w;
    long long p;             // output pixels n * ho * wo
    int stages;
    int blockdiag;           // grouped conv as block-diagonal GEMM: tile n0 reads channels [n0, n0 + 64) only
    // Strided output (one parity class of a strided backward-data pass): pixel (img, i, j) of the
    // class goes to out_strided + img out_sn + i out_sh + j out_sw (elements).  NULL: dense TMA stores.
    __nv_bfloat16 *out_strided;
    long long out_sn;
    int out_sh, out_sw;
    // Small-C_in ("stem") mode: the activation map is a 5-D window view {64, wo, ho, r, n} of a packed,
    // zero-bordered copy of X (8 channels per pixel; 8 pixels x 8 channels = one 128-byte K row per tap
    // row r), tiles are stem_th x stem_tw output patches (stem_th * stem_tw = 128), the output map is 4-D.
    int stem, stem_tw, stem_th, stem_tiles_w, stem_tiles_h;
    int resident;            // 1: the CTA's whole weight slab [BN][K] stays in shared memory (loaded once)
    int f16;                 // 16-bit storage type: 0 bf16, 1 IEEE half
    BnFold fold;             // fold.gamma != NULL: scale and shift formed in the kernel from the BN parameters
};

struct ConvSmemCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];     // MMA issuer -> epilogue, one per accumulator buffer
    uint64_t tmem_empty[2];    // epilogue -> MMA issuer (4 arrivals: one per epilogue warp)
    uint64_t bfull;            // resident weight slab has landed
    uint32_t tmem_base;
    int abort_flag;
};

// Persistent: CTA b works on tiles b, b + gridDim.x, ...; tile t covers output pixels
// [128 (t / n_tiles), +128) and output channels [BN (t % n_tiles), +BN).  The accumulator is
// double-buffered in tensor memory (2 x BN columns), so the MMAs of a tile overlap the epilogue of
// the tile before, and the TMA ring runs ahead across tile boundaries.
template <int BN>
__global__ void __launch_bounds__(kConvThreads) umma_conv_kernel(const __grid_constant__ CUtensorMap tm_act,
                                                                const __grid_constant__ CUtensorMap tm_w,
                                                                const __grid_constant__ CUtensorMap tm_out,
                                                                const ConvGemm g, const float *__restrict__ bias,
                                                                int *err) {
    extern __shared__ uint8_t smem_raw[];
    constexpr uint32_t kABytes = kBM * kBK * 2, kBBytes = BN * kBK * 2;
    const int cchunks = g.blockdiag ? 1 : g.ca / kBK;
    const int num_kb = g.taps_h * g.taps_w * cchunks;
    // Ring slots hold the activation tile and, unless the weights are resident, the weight tile.
    const uint32_t kStageBytes = g.resident ? kABytes : kABytes + kBBytes;
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *slab = tiles + (size_t)g.stages * kStageBytes;            // resident weights: num_kb x [BN][64]
    uint8_t *staging = slab + (g.resident ? (size_t)num_kb * kBBytes : 0);   // 8 warps x 2 x [32 rows][128 B]
    ConvSmemCtl *ctl = (ConvSmemCtl *)(staging + kStagingBytes);
    float *bias_s = (float *)(((uintptr_t)(ctl + 1) + 15) & ~(uintptr_t)15);   // cn floats
    float *scale_s = bias_s + g.cn;                                            // cn floats (fold mode)
    const bool fold = g.fold.gamma != nullptr;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = g.stages;
    const uint32_t n_tiles = (uint32_t)(g.cn + BN - 1) / BN;
    const uint32_t m_tiles = (uint32_t)((g.p + kBM - 1) / kBM);
    const uint32_t total_tiles = m_tiles * n_tiles;
    // Tile i of this CTA.  Resident weights: the CTA keeps one n-tile (blockIdx.x % n_tiles) and walks
    // m-tiles; otherwise tiles are dealt round-robin with the n-tiles of an m-tile on neighbouring CTAs.
    auto tile_of = [&](uint32_t i, uint32_t &mt, uint32_t &nt) -> bool {
        if (g.resident) {
            nt = blockIdx.x % n_tiles;
            mt = blockIdx.x / n_tiles + i * (gridDim.x / n_tiles);
            return mt < m_tiles;
        }
        const uint32_t t = blockIdx.x + i * gridDim.x;
        if (t >= total_tiles) return false;
        mt = t / n_tiles;
        nt = t - mt * n_tiles;
        return true;
    };
    volatile int *abort_flag = &ctl->abort_flag;

    if (threadIdx.x == 0) {
        CONVBN_TRACE_POINT(0);
        for (int s = 0; s < stages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tmem_full[a], 1); mbar_init(&ctl->tmem_empty[a], 4); }
        mbar_init(&ctl->bfull, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, 2 * BN);
        tmem_relinquish();
    }
    // Everything above touched only this CTA's own shared / tensor memory.  Global memory (inputs that
    // an earlier kernel may still be writing, outputs it may still be reading) comes after this wait.
    // the tensor maps are kernel parameters, not data of an earlier kernel: fetch them before the wait
    if (threadIdx.x == 0) { prefetch_tensormap(&tm_act); prefetch_tensormap(&tm_w); prefetch_tensormap(&tm_out); }
    pdl_wait();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(1);
    if (fold) {
        // On-the-fly reparameterisation (Sec. 3.3 / 3.4): s = gamma / sqrt(var + eps), b' = (b - mu) s + beta.
        // s multiplies the fp32 accumulator (the associative law of Sec. 3.2.2), so omega is used unrounded.
        for (int c = threadIdx.x; c < g.cn; c += kConvThreads) {
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
        for (int c = threadIdx.x; c < g.cn; c += kConvThreads) bias_s[c] = bias[c];
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
    const uint32_t tmem_base = ctl->tmem_base;
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(2);

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // The whole warp runs the loop; lane 0 arms the barrier and loads the activation tile, lane 1
        // loads the weight tile, so the two copies are issued in parallel.
        uint32_t it = 0;                         // k-blocks issued so far
        int s = 0;                               // ring slot and its phase, advanced incrementally
        uint32_t ph = 0;
        bool ok = true;
        if (g.resident && lane == 1) {
            const int n0 = (int)(blockIdx.x % n_tiles) * BN;
            mbar_arrive_expect_tx(&ctl->bfull, (uint32_t)num_kb * kBBytes);
            for (int kb = 0; kb < num_kb; ++kb) tma_load_2d(slab + (size_t)kb * kBBytes, &tm_w, &ctl->bfull, kb * kBK, n0);
        }
        uint32_t mt, nt;
        for (uint32_t i = 0; ok && tile_of(i, mt, nt); ++i) {
            // 32-bit arithmetic: 64-bit divisions would cost about a microsecond per tile here
            const uint32_t m0 = mt * kBM;
            const int n0 = (int)nt * BN;
            uint32_t tq, img;
            int wo0, ho0;
            if (g.stem) {       // m-tile -> (image, patch row, patch column)
                tq = mt / (uint32_t)g.stem_tiles_w;
                wo0 = (int)(mt - tq * (uint32_t)g.stem_tiles_w) * g.stem_tw;
                img = tq / (uint32_t)g.stem_tiles_h;
                ho0 = (int)(tq - img * (uint32_t)g.stem_tiles_h) * g.stem_th;
            } else {
                tq = m0 / (uint32_t)g.wo;
                wo0 = (int)(m0 - tq * (uint32_t)g.wo);
                img = tq / (uint32_t)g.ho;
                ho0 = (int)(tq - img * (uint32_t)g.ho);
            }
            const int img0 = (int)img;
            const int base_w = g.lower_w + wo0 * g.stride_w, base_h = g.lower_h + ho0 * g.stride_h;
            int r = 0, q = 0, cc = 0;
            for (int kb = 0; kb < num_kb; ++kb, ++it) {
                { CONVBN_TRACE_T0();
                ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag));
                if (lane == 0) CONVBN_TRACE_ACC(12); }
                if (!ok) break;
                uint8_t *a_dst = tiles + (size_t)s * kStageBytes, *b_dst = a_dst + kABytes;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&ctl->full[s], kStageBytes);   // (activation + weight tile) or activation only
                    if (g.stem)
                        tma_load_5d(a_dst, &tm_act, &ctl->full[s], 0, wo0, ho0, kb, img0);
                    else
                    tma_load_im2col_4d(a_dst, &tm_act, &ctl->full[s], (g.blockdiag ? n0 : 0) + cc * kBK, base_w, base_h, img0,
                                       (uint16_t)(q * g.dil_w), (uint16_t)(r * g.dil_h));
                } else if (lane == 1 && !g.resident) {
                    tma_load_2d(b_dst, &tm_w, &ctl->full[s], kb * kBK, n0);
                }
                if (++cc == cchunks) { cc = 0; if (++q == g.taps_w) { q = 0; ++r; } }
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
        }
        if (!ok && lane == 0) {
            atomicOr(err, ERRW_TIMEOUT);
            ctl->abort_flag = 1;
            // Let the copies already issued land (bounded) before the CTA may exit.
            const uint32_t first = it > (uint32_t)stages ? it - stages : 0;
            for (uint32_t j = first; j < it; ++j)
                mbar_wait_bounded(&ctl->full[j % stages], (j / stages) & 1u, nullptr, 200000000ull);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            const uint32_t idesc = idesc_h16_f32(kBM, BN, 0, 0, g.f16);
            const uint32_t hi = smem_desc_hi_sw128(1024);
            const uint32_t tiles_lo = smem_desc_lo(smem_u32(tiles), 16), slab_lo = smem_desc_lo(smem_u32(slab), 16);
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (g.resident) {
                ok = mbar_wait_bounded(&ctl->bfull, 0, abort_flag);
                tc_fence_after_sync();
            }
            uint32_t mt, nt;
            for (uint32_t i = 0; ok && tile_of(i, mt, nt); ++i) {
                const uint32_t acc = i & 1u;
                { CONVBN_TRACE_T0();
                if (!mbar_wait_bounded(&ctl->tmem_empty[acc], ((i >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                CONVBN_TRACE_ACC(13); }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    { CONVBN_TRACE_T0();
                    if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
                    CONVBN_TRACE_ACC(14); }
                    if (i == 0 && kb == 0) CONVBN_TRACE_POINT(4);
                    tc_fence_after_sync();
                    // descriptors as halves: only the start-address field (16-byte units) moves
                    const uint32_t a_lo = tiles_lo + (uint32_t)s * (kStageBytes >> 4);
                    const uint32_t b_lo = g.resident ? slab_lo + (uint32_t)kb * (kBBytes >> 4) : a_lo + (kABytes >> 4);
                    if (kb == 0) umma_bf16_ss_halves<false>(d_tmem, a_lo, hi, b_lo, hi, idesc);
                    else umma_bf16_ss_halves<true>(d_tmem, a_lo, hi, b_lo, hi, idesc);
#pragma unroll
                    for (int k = 1; k < kBK / kUmmaK; ++k)
                        umma_bf16_ss_halves<true>(d_tmem, a_lo + (uint32_t)k * 2u, hi, b_lo + (uint32_t)k * 2u, hi, idesc);
                    umma_commit(&ctl->empty[s]);
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(&ctl->tmem_full[acc]);
                CONVBN_TRACE_POINT(6);
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else {
        // ---------------- epilogue: tensor memory -> registers -> bf16 -> shared -> TMA store --------
        // Two groups of four warps; group e drains accumulator buffer e, i.e. every other tile of this
        // CTA, so two tiles are in their epilogue at once.  Each warp owns 32 accumulator rows and two
        // private [32 rows][64 columns] staging buffers (128-byte swizzle): warp-level sync only.
        const int quarter = warp & 3;                      // tensor-memory lanes this warp may read
        const uint32_t egroup = (uint32_t)(warp - 2) >> 2; // 0: warps 2-5, 1: warps 6-9
        uint8_t *stage_buf = staging + (size_t)(warp - 2) * kStagingWarpBytes;
        uint32_t mt, nt;
        for (uint32_t i = egroup; tile_of(i, mt, nt); i += 2) {
            const uint32_t acc = egroup;
            CONVBN_TRACE_T0();
            const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->tmem_full[acc], (i >> 1) & 1u, abort_flag));
            if (warp == 2 && lane == 0) CONVBN_TRACE_ACC(15);
            if (!ok) {
                if (lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
                break;
            }
            tc_fence_after_sync();
            const uint32_t m0 = mt * kBM;
            const int n0 = (int)nt * BN;
            const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(quarter * 32) << 16);
            int ncols = g.cn - n0;                          // valid columns of this tile
            if (ncols > BN) ncols = BN;
            __nv_bfloat16 *srow = nullptr;                  // strided mode: this thread's output pixel
            if (g.out_strided) {
                const uint32_t m = m0 + quarter * 32 + lane;
                if ((long long)m < g.p) {
                    const uint32_t tq = m / (uint32_t)g.wo, img = tq / (uint32_t)g.ho;
                    srow = g.out_strided + (size_t)img * g.out_sn + (size_t)(tq - img * (uint32_t)g.ho) * g.out_sh +
                           (size_t)(m - tq * (uint32_t)g.wo) * g.out_sw + n0;
                }
            }
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 64) {
                uint32_t v[64];
                if (c0 < ncols) {
                    tmem_ld_32x32(t_row + (uint32_t)c0, *(uint32_t(*)[32]) & v[0]);
                    tmem_ld_32x32(t_row + (uint32_t)c0 + 32, *(uint32_t(*)[32]) & v[32]);
                    tmem_ld_wait();
                }
                if (c0 + 64 >= BN) {
                    // every column of this accumulator has been read: hand the buffer back
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->tmem_empty[acc]);
                }
                if (c0 < ncols && g.out_strided) {
                    if (srow) {
#pragma unroll
                        for (int j = 0; j < 64; j += 8) {
                            if (c0 + j < ncols) {
                                uint4 pk;
                                pk.x = pack2_h16(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), g.f16);
                                pk.y = pack2_h16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]), g.f16);
                                pk.z = pack2_h16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]), g.f16);
                                pk.w = pack2_h16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]), g.f16);
                                *(uint4 *)(srow + c0 + j) = pk;
                            }
                        }
                    }
                } else if (c0 < ncols) {
                    uint8_t *buf = stage_buf;
                    // the previous store read this buffer: wait until it no longer does (shared memory
                    // is better spent on ring slots than on a second staging buffer)
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
                    uint8_t *row = buf + lane * 128;
                    auto pack_rows = [&](auto half_tag) {
                        constexpr bool H = decltype(half_tag)::value;
    #pragma unroll
                        for (int j = 0; j < 64; j += 8) {
                            float f[8];
    #pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[j + e]);
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
                            uint4 pk;
                            pk.x = pack2_t<H>(f[0], f[1]);
                            pk.y = pack2_t<H>(f[2], f[3]);
                            pk.z = pack2_t<H>(f[4], f[5]);
                            pk.w = pack2_t<H>(f[6], f[7]);
                            *(uint4 *)(row + ((((j >> 3) ^ (lane & 7)) & 7) << 4)) = pk;
                        }
                    };
                    if (g.f16) pack_rows(std::true_type{}); else pack_rows(std::false_type{});
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (g.stem) {
                            // this warp's 32 accumulator rows are (32 / stem_tw) patch rows of stem_tw pixels
                            const uint32_t tq2 = mt / (uint32_t)g.stem_tiles_w, im2 = tq2 / (uint32_t)g.stem_tiles_h;
                            tma_store_4d(&tm_out, buf, n0 + c0, (int)(mt - tq2 * (uint32_t)g.stem_tiles_w) * g.stem_tw,
                                         (int)(tq2 - im2 * (uint32_t)g.stem_tiles_h) * g.stem_th + quarter * (32 / g.stem_tw),
                                         (int)im2);
                        } else {
                            tma_store_2d(&tm_out, buf, n0 + c0, (int)(m0 + quarter * 32));
                        }
                        tma_store_commit();
                    }
                }
            }
        }
        if (warp == 2 && lane == 0) CONVBN_TRACE_POINT(9);
        if (lane == 0) tma_store_wait_all<0>();             // global writes done before the CTA exits
        if (warp == 2 && lane == 0) CONVBN_TRACE_POINT(10);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) CONVBN_TRACE_POINT(11);
    if (warp == 1) tmem_dealloc(tmem_base, 2 * BN);
}

// ---- failure-path self-test: the bounded wait of the kernels above, on a barrier nobody completes --------
__global__ void selftest_wait_timeout_kernel(unsigned long long limit_ns, int *err) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        if (!mbar_wait_bounded(&bar, 0, nullptr, limit_ns)) atomicOr(err, ERRW_TIMEOUT);
    }
}

cudaError_t launch_selftest_wait_timeout(unsigned long long limit_ns, cudaStream_t st) {
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    selftest_wait_timeout_kernel<<<1, 32, 0, st>>>(limit_ns, err);
    return cudaGetLastError();
}

// ---- host side: tensor maps and launch ---------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;
std::once_flag g_encode_once;

bool load_encoders() {
    std::call_once(g_encode_once, [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode_tiled = (EncodeTiledFn)f;
        f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode_im2col = (EncodeIm2colFn)f;
    });
    return g_encode_tiled && g_encode_im2col;
}

}  // namespace

// bf16 row-major matrix [rows][cols] -> box of box_rows x 64 columns, 128-byte swizzle.
bool make_tmap_matrix_bf16(CUtensorMap *tm, const void *base, long long rows, long long cols, int box_rows,
                           int box_cols) {
    if (!load_encoders()) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// NHWC bf16 tensor [n][h][w][c] -> im2col-mode map: `pixels` consecutive output positions x 64 channels
// per load, 128-byte swizzle, zero fill outside the image.
bool make_tmap_im2col_bf16(CUtensorMap *tm, const void *base, int n, int h, int w, int c, int lower_h,
                           int lower_w, int upper_h, int upper_w, int stride_h, int stride_w, int pixels,
                           int channels) {
    if (!load_encoders()) return false;
    cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t strides[3] = {(cuuint64_t)c * 2, (cuuint64_t)w * c * 2, (cuuint64_t)h * w * c * 2};
    int lower[2] = {lower_w, lower_h};
    int upper[2] = {upper_w, upper_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride_w, (cuuint32_t)stride_h, 1};
    return g_encode_im2col(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, lower,
                           upper, (cuuint32_t)channels, (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool encode_tiled_bf16(CUtensorMap *tm, const void *base, int rank, const unsigned long long *dims,
                              const unsigned long long *strides_bytes, const unsigned int *box, CUtensorMapSwizzle sw) {
    if (!load_encoders() || rank < 1 || rank > 5) return false;
    cuuint64_t d[5], st[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 1; i < rank; ++i) st[i - 1] = strides_bytes[i];
    return g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), d, st, bx,
                          es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_tiled_bf16(CUtensorMap *tm, const void *base, int rank, const unsigned long long *dims,
                          const unsigned long long *strides_bytes, const unsigned int *box) {
    return encode_tiled_bf16(tm, base, rank, dims, strides_bytes, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

bool make_tmap_tiled_bf16_linear(CUtensorMap *tm, const void *base, int rank, const unsigned long long *dims,
                                 const unsigned long long *strides_bytes, const unsigned int *box) {
    return encode_tiled_bf16(tm, base, rank, dims, strides_bytes, box, CU_TENSOR_MAP_SWIZZLE_NONE);
}

bool umma_conv_eligible(const UmmaConvShape &s) {
    if (s.ca % kBK || s.cn % 8 || s.cn < 64 || s.cn > 4096) return false;
    if (s.blockdiag && (s.ca != s.cn)) return false;
    if (s.lower_h < -128 || s.lower_h > 127 || s.lower_w < -128 || s.lower_w > 127) return false;
    if ((s.taps_h - 1) * s.dil_h > 255 || (s.taps_w - 1) * s.dil_w > 255) return false;
    if (s.stride_h > 8 || s.stride_w > 8) return false;
    if ((long long)s.taps_h * s.taps_w * s.ca > (1 << 24)) return false;
    if ((long long)s.n * s.ho * s.wo >= (1LL << 31) - 256) return false;
    return true;
}

static int sm_count() { return device_sm_count(); }

template <int BN>
static cudaError_t launch_bn(const CUtensorMap &ta, const CUtensorMap &tw, const CUtensorMap &tout, ConvGemm g,
                             const float *bias, int *err, cudaStream_t st) {
    const size_t a_bytes = (size_t)kBM * kBK * 2, b_bytes = (size_t)BN * kBK * 2;
    size_t fixed = 1024 + kStagingBytes + sizeof(ConvSmemCtl) + 2 * (size_t)g.cn * sizeof(float) + 16;
    const int num_kb = g.taps_h * g.taps_w * (g.blockdiag ? 1 : g.ca / kBK);
    const long long m_tiles = (g.p + kBM - 1) / kBM, n_tiles = (g.cn + BN - 1) / BN;
    long long grid_l = m_tiles * n_tiles < sm_count() ? m_tiles * n_tiles : sm_count();
    // Weights stay resident when the CTA's slab fits beside at least four activation slots and the
    // grid can give every CTA one fixed n-tile.
    const size_t slab = (size_t)num_kb * b_bytes;
    g.resident = 0;
    if (slab <= 104 * 1024 && fixed + slab + 4 * a_bytes <= 220 * 1024 && m_tiles * n_tiles >= sm_count() &&
        n_tiles <= sm_count()) {
        g.resident = 1;
        grid_l = sm_count() - sm_count() % n_tiles;
        fixed += slab;
    }
    const size_t stage = g.resident ? a_bytes : a_bytes + b_bytes;
    int stages = (int)((220 * 1024 - fixed) / stage);  // one CTA per SM owns the shared memory
    if (stages > kMaxStages) stages = kMaxStages;
    g.stages = stages;
    const size_t smem = stages * stage + fixed;
    static PerDevice attr_done;
    if (cudaError_t e = max_dynamic_smem_once(umma_conv_kernel<BN>, 224 * 1024, &attr_done); e != cudaSuccess) return e;
    static PerDevice carve;
    prefer_max_shared_once(umma_conv_kernel<BN>, &carve);
    const unsigned grid = (unsigned)grid_l;
    return launch_pdl(umma_conv_kernel<BN>, dim3(grid), dim3(kConvThreads), smem, st, ta, tw, tout, g, bias, err);
}

// Tile width: fewest rounds of tiles over the SMs, weighted by the time of one tile (N = 64 tiles are
// bound by shared-memory operand bandwidth, about 1.5x slower per column than wider ones).
static int pick_bn(long long tiles_m, int cn) {
    int best = 64;
    double best_cost = 1e30;
    const int cand[3] = {256, 128, 64};
    for (int c = 0; c < 3; ++c) {
        const int bn = cand[c];
        if (bn > 64 && cn <= bn / 2) continue;
        const long long tiles = tiles_m * ((cn + bn - 1) / bn);
        const long long rounds = (tiles + sm_count() - 1) / sm_count();
        const double cost = (double)rounds * bn * (bn == 64 ? 1.5 : 1.0);
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

cudaError_t launch_umma_conv(const UmmaConvShape &s, const void *act, const void *wmat, const float *bias,
                             void *out, cudaStream_t st, const BnFold *fold) {
    ConvGemm g;
    g.ho = s.ho; g.wo = s.wo; g.cn = s.cn; g.ca = s.ca; g.taps_h = s.taps_h; g.taps_w = s.taps_w;
    g.lower_h = s.lower_h; g.lower_w = s.lower_w; g.stride_h = s.stride_h; g.stride_w = s.stride_w;
    g.dil_h = s.dil_h; g.dil_w = s.dil_w; g.p = (long long)s.n * s.ho * s.wo; g.stages = 1;
    g.blockdiag = s.blockdiag;
    g.f16 = call_f16();
    g.stem = 0; g.stem_tw = g.stem_th = g.stem_tiles_w = g.stem_tiles_h = 1;
    g.fold = fold ? *fold : BnFold{nullptr, nullptr, nullptr, nullptr, nullptr, 0.f, nullptr};
    g.out_strided = s.out_sw ? (__nv_bfloat16 *)out : nullptr;
    g.out_sn = s.out_sn; g.out_sh = s.out_sh; g.out_sw = s.out_sw;
    // The bounding box of base pixels has ho x wo positions: upper = lower + (out-1) stride - (in-1).
    const int upper_h = s.lower_h + (s.ho - 1) * s.stride_h - (s.ha - 1);
    const int upper_w = s.lower_w + (s.wo - 1) * s.stride_w - (s.wa - 1);
    const long long tiles_m = (g.p + kBM - 1) / kBM;
    const int bn = s.blockdiag ? 64 : pick_bn(tiles_m, s.cn);
    CUtensorMap ta, tw, tout;
    // (in strided mode the output map is encoded but never used: every row is stored by its thread)
    if (!make_tmap_matrix_bf16(&tout, out, s.out_sw ? 32 : g.p, s.cn, 32, 64)) return cudaErrorInvalidValue;
    if (!make_tmap_im2col_bf16(&ta, act, s.n, s.ha, s.wa, s.ca, s.lower_h, s.lower_w, upper_h, upper_w, s.stride_h,
                               s.stride_w, kBM, kBK))
        return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tw, wmat, s.cn, (long long)s.taps_h * s.taps_w * (s.blockdiag ? 64 : s.ca), bn, kBK))
        return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    if (bn == 64) return launch_bn<64>(ta, tw, tout, g, bias, err, st);
    if (bn == 128) return launch_bn<128>(ta, tw, tout, g, bias, err, st);
    return launch_bn<256>(ta, tw, tout, g, bias, err, st);
}

// Forward pass of a small-C_in layer on the packed input (see stem_kernels.cu): tiles of 8 x 16 output
// pixels, K = stem_krows rows of 64, weights resident.
cudaError_t launch_stem_fwd(const Problem &pb, const void *x_packed, const void *wst, const float *bias, void *out,
                            cudaStream_t st, const BnFold *fold) {
    const int krows = stem_krows(pb);
    ConvGemm g;
    g.ho = pb.h_out; g.wo = pb.w_out; g.cn = pb.c_out; g.ca = 64; g.taps_h = krows; g.taps_w = 1;
    g.lower_h = g.lower_w = 0; g.stride_h = g.stride_w = g.dil_h = g.dil_w = 1;
    g.stem = 1; g.stem_tw = 16; g.stem_th = 8;
    g.stem_tiles_w = (pb.w_out + 15) / 16; g.stem_tiles_h = (pb.h_out + 7) / 8;
    g.p = (long long)pb.n * g.stem_tiles_h * g.stem_tiles_w * kBM;      // m-tiles x 128 (patches, ragged edges clipped)
    g.stages = 1; g.blockdiag = 0; g.out_strided = nullptr; g.out_sn = 0; g.out_sh = g.out_sw = 0;
    g.f16 = call_f16();
    g.fold = fold ? *fold : BnFold{nullptr, nullptr, nullptr, nullptr, nullptr, 0.f, nullptr};
    CUtensorMap ta, tw, tout;
    {   // overlapping windows: 64 elements (8 pixels x 8 channels) starting at every output column
        const unsigned long long dims[5] = {64, (unsigned long long)pb.w_out, (unsigned long long)pb.h_out,
                                            (unsigned long long)krows, (unsigned long long)pb.n};
        unsigned long long str[5];
        stem_window_strides(pb, str);
        const unsigned int box[5] = {64, 16, 8, 1, 1};
        if (!make_tmap_tiled_bf16(&ta, x_packed, 5, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const unsigned long long dims[4] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                            (unsigned long long)pb.h_out, (unsigned long long)pb.n};
        const unsigned long long str[4] = {0, (unsigned long long)pb.c_out * 2,
                                           (unsigned long long)pb.w_out * pb.c_out * 2,
                                           (unsigned long long)pb.h_out * pb.w_out * pb.c_out * 2};
        const unsigned int box[4] = {64, 16, 2, 1};
        if (!make_tmap_tiled_bf16(&tout, out, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    if (!make_tmap_matrix_bf16(&tw, wst, pb.c_out, (long long)krows * 64, 64, kBK)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    return launch_bn<64>(ta, tw, tout, g, bias, err, st);
}

}  // namespace convbn
