// Fused backward pass of a 1x1, stride-1 ConvBN block in Tune mode (Table 2, Tune row; Sec. 3.2.1):
//     dX      = dZ omega'                      (omega' = s omega, formed in shared memory, never stored)
//     domega' = dZ^T X       sum dZ            (fp32 partial per CTA, finished by the fused epilogue kernel)
// dZ is read from memory ONCE: the same shared-memory tile [128 pixels][C_out] is the K-major A operand of the
// data-gradient GEMM and an MN-major operand of the weight-gradient GEMM, next to the X tile [128 pixels][C_in].
// Two shapes of layer are served, the bottleneck's 1x1 convolutions:
//   WIDE_IN  (C_in  = 128 or 256, C_out = 64): domega' accumulates as [ci][co]  (A = X tile, B = dZ tile),
//            sum dZ from one more MMA whose A operand is a tile of ones;
//   WIDE_OUT (C_out = 128 or 256, C_in  = 64): domega' accumulates as [co][ci]  (A = dZ tile, B = X tile),
//            sum dZ from one more MMA whose B operand is a tile of ones (16 columns).
// A CTA owns a contiguous range of 128-pixel tiles; its weight-gradient accumulators stay in tensor memory for
// the whole range.  Warps: 0 TMA producer, 1 MMA issuer and tensor-memory owner, 2-9 epilogue (dX tiles:
// tensor memory -> bf16 -> swizzled staging -> TMA store; at the end the partial of domega').
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace convbn {

using namespace ptx;

constexpr int kFbThreads = 320;
constexpr int kFbStages = 2;
constexpr uint32_t kFbBox = 128 * 128;        // one [128 pixels][64 channels] bf16 box

struct FusedBwd {
    long long p;            // pixels
    int m_tiles;            // ceil(p / 128)
    const float *vec3;      // saved [s | b' | r]
    int f16;                // 16-bit storage type: 0 bf16, 1 IEEE half
};

struct FbCtl {
    uint64_t full[kFbStages], empty[kFbStages];
    uint64_t dx_full[2], dx_empty[2];
    uint64_t acc_done;
    uint32_t tmem_base;
    int abort_flag;
};

template <int CI, int CO>
struct FbShape {
    static constexpr bool kWideIn = CI >= CO;
    static constexpr int kXBoxes = CI / 64, kDzBoxes = CO / 64;
    static constexpr uint32_t kStageBytes = (uint32_t)(kXBoxes + kDzBoxes) * kFbBox;
    static constexpr int kDxBufs = CI <= 128 ? 2 : 1;                    // dX accumulators [128][CI]
    static constexpr int kDxCols = CI * kDxBufs;
    static constexpr int kWide = kWideIn ? CI : CO, kNarrow = kWideIn ? CO : CI;
    static constexpr int kMBlocks = kWide / 128;                         // weight-gradient M blocks
    static constexpr int kDwCol0 = kDxCols;                              // [kWide][kNarrow] accumulators
    static constexpr int kSumCol0 = kDwCol0 + kMBlocks * kNarrow;
    static constexpr int kSumCols = kWideIn ? CO : 16 * kMBlocks;
    static_assert(kSumCol0 + kSumCols <= 512, "tensor memory");
    static_assert((CI == 64) != (CO == 64) && kWide % 128 == 0 && kWide <= 256, "supported channel counts");
};

template <int CI, int CO>
__global__ void __launch_bounds__(kFbThreads) fused_bwd1x1_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                                 const __grid_constant__ CUtensorMap tm_x,
                                                                 const __grid_constant__ CUtensorMap tm_dx,
                                                                 const FusedBwd g, const __nv_bfloat16 *__restrict__ w,
                                                                 float *__restrict__ partials, float *__restrict__ bsum,
                                                                 unsigned int *__restrict__ counters, int ncounters,
                                                                 int *err) {
    using S = FbShape<CI, CO>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *stages = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *wres = stages + (size_t)kFbStages * S::kStageBytes;     // omega' as [ci / 64][co][64 ci], swizzled
    uint8_t *ones = wres + (size_t)CI * CO * 2;                      // 8 rows of 64 bf16 1.0 (read with all strides 0)
    uint8_t *staging = ones + 1024;                                  // 8 warps x [32 rows][128 B]
    FbCtl *ctl = (FbCtl *)(staging + 8 * 4096);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &ctl->abort_flag;
    const int tile_lo = (int)((long long)g.m_tiles * blockIdx.x / gridDim.x);
    const int tile_hi = (int)((long long)g.m_tiles * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFbStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&ctl->dx_full[s], 1); mbar_init(&ctl->dx_empty[s], S::kDxBufs == 2 ? 4 : 8); }
        mbar_init(&ctl->acc_done, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_dz); prefetch_tensormap(&tm_x); prefetch_tensormap(&tm_dx);
    }
    if (warp == 1) {
        tmem_alloc(&ctl->tmem_base, 512);
        tmem_relinquish();
    }
    {
        const uint32_t one2 = one_h16(g.f16) * 0x10001u;
        const uint4 one4 = make_uint4(one2, one2, one2, one2);
        for (int i = threadIdx.x; i < 1024 / 16; i += kFbThreads) ((uint4 *)ones)[i] = one4;
    }
    pdl_wait();
    if (counters && blockIdx.x == 0)
        for (int i = threadIdx.x; i < ncounters; i += kFbThreads) counters[i] = 0u;
    // omega' = s omega (Sec. 3.3), one rounding to bf16, laid out as the MN-major B operand of the data-gradient
    // GEMM: K = co rows of 128 bytes (64 ci), 128-byte swizzle, one block per 64 input channels
    for (int i = threadIdx.x; i < CO * (CI / 8); i += kFbThreads) {
        const int co = i / (CI / 8), c8 = i - co * (CI / 8), ci = c8 * 8;
        const float sc = g.vec3[co];
        const uint4 raw = __ldg((const uint4 *)(w + (size_t)co * CI + ci));
        const uint32_t in[4] = {raw.x, raw.y, raw.z, raw.w};
        uint32_t out[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const float lo = unpack_h16((uint16_t)(in[h] & 0xFFFFu), g.f16) * sc, hi = unpack_h16((uint16_t)(in[h] >> 16), g.f16) * sc;
            out[h] = pack2_h16(lo, hi, g.f16);
        }
        *(uint4 *)(wres + (size_t)(ci >> 6) * (CO * 128) + co * 128 + (((((ci & 63) >> 3) ^ (co & 7)) & 7) << 4)) =
            make_uint4(out[0], out[1], out[2], out[3]);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();       // only now: this CTA owns its tensor-memory columns
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ---------------- producer: the dZ boxes, then the X boxes of a tile ----------------
        int s = 0, issued = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int t = tile_lo; t < tile_hi; ++t) {
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag));
            if (!ok) break;
            uint8_t *dst = stages + (size_t)s * S::kStageBytes;
            if (lane == 0) mbar_arrive_expect_tx(&ctl->full[s], S::kStageBytes);
            __syncwarp();
            if (lane < S::kDzBoxes) tma_load_2d(dst + (size_t)lane * kFbBox, &tm_dz, &ctl->full[s], lane * 64, t * 128);
            else if (lane < S::kDzBoxes + S::kXBoxes)
                tma_load_2d(dst + (size_t)lane * kFbBox, &tm_x, &ctl->full[s], (lane - S::kDzBoxes) * 64, t * 128);
            ++issued;
            if (++s == kFbStages) { s = 0; ph ^= 1u; }
        }
        if (!ok && lane == 0) {
            atomicOr(err, ERRW_TIMEOUT);
            ctl->abort_flag = 1;
            for (int j = issued > kFbStages ? issued - kFbStages : 0; j < issued; ++j)
                mbar_wait_bounded(&ctl->full[j % kFbStages], (uint32_t)(j / kFbStages) & 1u, nullptr, 200000000ull);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            const uint32_t hi = smem_desc_hi_sw128(1024);
            constexpr uint32_t kBox16 = kFbBox >> 4;
            const uint32_t idesc_dx = idesc_h16_f32(128, CI, 0, 1, g.f16);          // A = dZ (K-major), B = omega' (MN-major)
            const uint32_t idesc_dw = idesc_h16_f32(128, S::kNarrow, 1, 1, g.f16);  // both operands MN-major
            const uint32_t idesc_sum = idesc_h16_f32(128, S::kWideIn ? CO : 16, 1, 1, g.f16);
            const uint32_t w_lo = smem_desc_lo(smem_u32(wres), CO * 128);           // N blocks CO * 128 bytes apart
            // a tile of ones of any extent: one 8 x 128-byte group, block stride 0, row-group stride 0
            const uint32_t ones_lo = smem_desc_lo(smem_u32(ones), 0), ones_hi = smem_desc_hi_sw128(0);
            int s = 0;
            uint32_t ph = 0, i = 0;
            bool ok = true;
            for (int t = tile_lo; t < tile_hi && ok; ++t, ++i) {
                if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
                const uint32_t buf = S::kDxBufs == 2 ? (i & 1u) : 0u, use = S::kDxBufs == 2 ? (i >> 1) : i;
                if (!mbar_wait_bounded(&ctl->dx_empty[buf], (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t st_addr = smem_u32(stages + (size_t)s * S::kStageBytes);
                const uint32_t dz_k = smem_desc_lo(st_addr, 16);                                   // K-major view
                const uint32_t dz_mn = smem_desc_lo(st_addr, kFbBox);                              // MN-major view
                const uint32_t x_mn = smem_desc_lo(st_addr + (uint32_t)S::kDzBoxes * kFbBox, kFbBox);
                // dX tile = dZ tile x omega': K = C_out in steps of 16
                const uint32_t d_dx = tmem_base + buf * (uint32_t)CI;
#pragma unroll
                for (int kk = 0; kk < CO / 16; ++kk) {
                    const uint32_t a_lo = dz_k + (uint32_t)(kk >> 2) * kBox16 + (uint32_t)(kk & 3) * 2u;
                    const uint32_t b_lo = w_lo + (uint32_t)kk * 128u;              // 16 rows of 128 bytes
                    if (kk == 0) umma_bf16_ss_halves<false>(d_dx, a_lo, hi, b_lo, hi, idesc_dx);
                    else umma_bf16_ss_halves<true>(d_dx, a_lo, hi, b_lo, hi, idesc_dx);
                }
                umma_commit(&ctl->dx_full[buf]);
                // domega' and sum dZ: K = the tile's 128 pixels in steps of 16 (two groups of 8 rows, 2048 bytes)
#pragma unroll 1
                for (int kt = 0; kt < 8; ++kt) {
                    const uint32_t koff = (uint32_t)kt * 128u;
#pragma unroll
                    for (int mb = 0; mb < S::kMBlocks; ++mb) {
                        const uint32_t d = tmem_base + (uint32_t)(S::kDwCol0 + mb * S::kNarrow);
                        const uint32_t a_lo = (S::kWideIn ? x_mn : dz_mn) + (uint32_t)(2 * mb) * kBox16 + koff;
                        const uint32_t b_lo = (S::kWideIn ? dz_mn : x_mn) + koff;
                        if (i == 0 && kt == 0) umma_bf16_ss_halves<false>(d, a_lo, hi, b_lo, hi, idesc_dw);
                        else umma_bf16_ss_halves<true>(d, a_lo, hi, b_lo, hi, idesc_dw);
                        if (!S::kWideIn) {
                            const uint32_t ds = tmem_base + (uint32_t)(S::kSumCol0 + mb * 16);
                            if (i == 0 && kt == 0) umma_bf16_ss_halves<false>(ds, a_lo, hi, ones_lo, ones_hi, idesc_sum);
                            else umma_bf16_ss_halves<true>(ds, a_lo, hi, ones_lo, ones_hi, idesc_sum);
                        }
                    }
                    if (S::kWideIn) {
                        const uint32_t ds = tmem_base + (uint32_t)S::kSumCol0;
                        if (i == 0 && kt == 0) umma_bf16_ss_halves<false>(ds, ones_lo, ones_hi, dz_mn + koff, hi, idesc_sum);
                        else umma_bf16_ss_halves<true>(ds, ones_lo, ones_hi, dz_mn + koff, hi, idesc_sum);
                    }
                }
                umma_commit(&ctl->empty[s]);
                if (++s == kFbStages) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(&ctl->acc_done);
            else { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3, egroup = (warp - 2) >> 2;
        uint8_t *buf_s = staging + (size_t)(warp - 2) * 4096;
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        bool ok = true;
        uint32_t i = 0;
        for (int t = tile_lo; t < tile_hi && ok; ++t, ++i) {
            const uint32_t buf = S::kDxBufs == 2 ? (i & 1u) : 0u, use = S::kDxBufs == 2 ? (i >> 1) : i;
            if (S::kDxBufs == 2 && (int)buf != egroup) continue;        // the two groups take alternate tiles
            ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->dx_full[buf], use & 1u, abort_flag));
            if (!ok) break;
            tc_fence_after_sync();
            // one accumulator: the groups split its columns; two accumulators: a group drains all columns
            const int c_lo = S::kDxBufs == 2 ? 0 : egroup * (CI / 2), c_hi = S::kDxBufs == 2 ? CI : c_lo + CI / 2;
#pragma unroll 1
            for (int c0 = c_lo; c0 < c_hi; c0 += 64) {
                uint32_t v[64];
                const uint32_t taddr = tmem_base + buf * (uint32_t)CI + (uint32_t)c0 + lane_sel;
                tmem_ld_32x32(taddr, *(uint32_t(*)[32]) & v[0]);
                tmem_ld_32x32(taddr + 32, *(uint32_t(*)[32]) & v[32]);
                tmem_ld_wait();
                if (c0 + 64 >= c_hi) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->dx_empty[buf]);
                }
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
                uint8_t *row = buf_s + lane * 128;
                auto pack_rows = [&](auto half_tag) {
                    constexpr bool H = decltype(half_tag)::value;
    #pragma unroll
                    for (int j = 0; j < 64; j += 8) {
                        uint4 pk;
                        pk.x = pack2_t<H>(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                        pk.y = pack2_t<H>(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        pk.z = pack2_t<H>(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                        pk.w = pack2_t<H>(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                        *(uint4 *)(row + ((((j >> 3) ^ (lane & 7)) & 7) << 4)) = pk;
                    }
                };
                if (g.f16) pack_rows(std::true_type{}); else pack_rows(std::false_type{});
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tm_dx, buf_s, c0, t * 128 + quarter * 32);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
        // ---- the CTA's partial of domega' as part[cta][k = ci][co] and its row of sums of dZ ----
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->acc_done, 0, abort_flag));
        if (ok) {
            tc_fence_after_sync();
            float *part = partials + (size_t)blockIdx.x * CI * CO;
            if (S::kWideIn) {
                // accumulator row = ci (M block mb, lane), columns = co: each thread owns one k row of 64 floats
                for (int mb = egroup; mb < S::kMBlocks; mb += 2) {
                    float *orow = part + (size_t)(mb * 128 + quarter * 32 + lane) * CO;
#pragma unroll 1
                    for (int c0 = 0; c0 < CO; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_32x32(tmem_base + (uint32_t)(S::kDwCol0 + mb * CO + c0) + lane_sel, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; j += 4) *(uint4 *)(orow + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    }
                }
                if (warp == 2) {                               // every row of the sums tile is sum dZ: take this warp's first
                    float *brow = bsum + (size_t)blockIdx.x * CO;
#pragma unroll 1
                    for (int c0 = 0; c0 < CO; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_32x32(tmem_base + (uint32_t)(S::kSumCol0 + c0) + lane_sel, v);
                        tmem_ld_wait();
                        if (lane == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *(uint4 *)(brow + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        }
                    }
                }
            } else {
                // accumulator row = co, columns = ci (64): part[ci][co] is the transpose; 32 consecutive co per ci
                // row are written together (128 bytes), lane = co
                for (int mb = egroup; mb < S::kMBlocks; mb += 2) {
                    const int co = mb * 128 + quarter * 32 + lane;
#pragma unroll 1
                    for (int c0 = 0; c0 < CI; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_32x32(tmem_base + (uint32_t)(S::kDwCol0 + mb * CI + c0) + lane_sel, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) part[(size_t)(c0 + j) * CO + co] = __uint_as_float(v[j]);
                    }
                    uint32_t sv[16];
                    tmem_ld_32x16(tmem_base + (uint32_t)(S::kSumCol0 + mb * 16) + lane_sel, sv);
                    tmem_ld_wait();
                    bsum[(size_t)blockIdx.x * CO + co] = __uint_as_float(sv[0]);
                }
            }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

// ---- host side --------------------------------------------------------------------------------------
namespace {
template <int CI, int CO>
cudaError_t launch_fb(const CUtensorMap &tdz, const CUtensorMap &tx, const CUtensorMap &tdx, const FusedBwd &g, unsigned grid,
                      const void *w, float *partials, float *bsum, unsigned int *counters, int *err, cudaStream_t st) {
    using S = FbShape<CI, CO>;
    const size_t smem = 1024 + (size_t)kFbStages * S::kStageBytes + (size_t)CI * CO * 2 + 1024 + 8 * 4096 + sizeof(FbCtl) + 64;
    static PerDevice attr, carve;
    if (cudaError_t e = max_dynamic_smem_once(fused_bwd1x1_kernel<CI, CO>, 227 * 1024, &attr); e != cudaSuccess) return e;
    prefer_max_shared_once(fused_bwd1x1_kernel<CI, CO>, &carve);
    return launch_pdl(fused_bwd1x1_kernel<CI, CO>, dim3(grid), dim3(kFbThreads), smem, st, tdz, tx, tdx, g,
                      (const __nv_bfloat16 *)w, partials, bsum, counters, CO / 32, err);
}
}  // namespace

bool fused_bwd1x1_eligible(const Problem &pb) {
    if (pb.groups != 1 || pb.kh != 1 || pb.kw != 1 || pb.stride_h != 1 || pb.stride_w != 1 || pb.pad_h || pb.pad_w) return false;
    const bool shape = (pb.c_out == 64 && (pb.c_in == 128 || pb.c_in == 256)) || (pb.c_in == 64 && (pb.c_out == 128 || pb.c_out == 256));
    return shape && pb.p >= 128 * 4 && pb.p < (1LL << 30);
}

int fused_bwd1x1_ctas(const Problem &pb) {
    const long long tiles = (pb.p + 127) / 128, sms = device_sm_count();
    return (int)(tiles < sms ? tiles : sms);
}

cudaError_t launch_fused_bwd1x1(const Problem &pb, const void *dz, const void *x, const void *w, const float *vec3, void *dx,
                                float *partials, float *bsum, unsigned int *counters, cudaStream_t st) {
    if (!fused_bwd1x1_eligible(pb)) return cudaErrorInvalidValue;
    FusedBwd g;
    g.p = pb.p; g.m_tiles = (int)((pb.p + 127) / 128); g.vec3 = vec3; g.f16 = call_f16();
    CUtensorMap tdz, tx, tdx;
    if (!make_tmap_matrix_bf16(&tdz, dz, pb.p, pb.c_out, 128, 64)) return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tx, x, pb.p, pb.c_in, 128, 64)) return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tdx, dx, pb.p, pb.c_in, 32, 64)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)fused_bwd1x1_ctas(pb);
    if (pb.c_in == 256) return launch_fb<256, 64>(tdz, tx, tdx, g, grid, w, partials, bsum, counters, err, st);
    if (pb.c_in == 128) return launch_fb<128, 64>(tdz, tx, tdx, g, grid, w, partials, bsum, counters, err, st);
    if (pb.c_out == 256) return launch_fb<64, 256>(tdz, tx, tdx, g, grid, w, partials, bsum, counters, err, st);
    return launch_fb<64, 128>(tdz, tx, tdx, g, grid, w, partials, bsum, counters, err, st);
}

}  // namespace convbn
