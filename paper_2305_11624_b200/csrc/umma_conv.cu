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
constexpr int kMaxStages = 8;
constexpr int kConvThreads = 192;

struct ConvGemm {
    int ho, wo;              // output spatial extent
    int cn;                  // output channels (GEMM N)
    int ca;                  // activation channels (multiple of 64)
    int taps_h, taps_w;
    int lower_h, lower_w;    // input coordinate read by output (0,0) at tap (0,0)
    int stride_h, stride_w, dil_h, dil_w;
    long long p;             // output pixels n * ho * wo
    int stages;
};

struct ConvSmemCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint32_t tmem_base;
    int abort_flag;
};

template <int BN>
__global__ void __launch_bounds__(kConvThreads) umma_conv_kernel(const __grid_constant__ CUtensorMap tm_act,
                                                                const __grid_constant__ CUtensorMap tm_w,
                                                                const ConvGemm g, const float *__restrict__ bias,
                                                                __nv_bfloat16 *__restrict__ out, int *err) {
    extern __shared__ uint8_t smem_raw[];
    constexpr uint32_t kABytes = kBM * kBK * 2, kBBytes = BN * kBK * 2, kStageBytes = kABytes + kBBytes;
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    ConvSmemCtl *ctl = (ConvSmemCtl *)(tiles + (size_t)g.stages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = g.stages;
    const int cchunks = g.ca / kBK;
    const int num_kb = g.taps_h * g.taps_w * cchunks;
    const long long m0 = (long long)blockIdx.x * kBM;
    const int n0 = blockIdx.y * BN;
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
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            prefetch_tensormap(&tm_act);
            prefetch_tensormap(&tm_w);
            const int wo0 = (int)(m0 % g.wo);
            const long long t = m0 / g.wo;
            const int ho0 = (int)(t % g.ho), img0 = (int)(t / g.ho);
            const int base_w = g.lower_w + wo0 * g.stride_w, base_h = g.lower_h + ho0 * g.stride_h;
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % stages;
                const uint32_t ph = (uint32_t)(kb / stages) & 1u;
                if (!mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag)) {
                    atomicOr(err, ERRW_TIMEOUT);
                    ctl->abort_flag = 1;
                    break;
                }
                const int tap = kb / cchunks, cc = kb - tap * cchunks;
                const int r = tap / g.taps_w, q = tap - r * g.taps_w;
                uint8_t *a_dst = tiles + (size_t)s * kStageBytes, *b_dst = a_dst + kABytes;
                mbar_arrive_expect_tx(&ctl->full[s], kStageBytes);
                tma_load_im2col_4d(a_dst, &tm_act, &ctl->full[s], cc * kBK, base_w, base_h, img0,
                                   (uint16_t)(q * g.dil_w), (uint16_t)(r * g.dil_h));
                tma_load_2d(b_dst, &tm_w, &ctl->full[s], kb * kBK, n0);
                ++issued;
            }
            if (ctl->abort_flag) {
                // Let the copies already issued land (bounded) before the CTA may exit.
                const int first = issued > stages ? issued - stages : 0;
                for (int kb = first; kb < issued; ++kb)
                    mbar_wait_bounded(&ctl->full[kb % stages], (uint32_t)(kb / stages) & 1u, nullptr, 200000000ull);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            constexpr uint32_t idesc = idesc_bf16_f32(kBM, BN, 0, 0);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % stages;
                const uint32_t ph = (uint32_t)(kb / stages) & 1u;
                if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) {
                    atomicOr(err, ERRW_TIMEOUT);
                    ctl->abort_flag = 1;
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t a_addr = smem_u32(tiles + (size_t)s * kStageBytes), b_addr = a_addr + kABytes;
#pragma unroll
                for (int k = 0; k < kBK / kUmmaK; ++k) {
                    const uint64_t ad = smem_desc_sw128(a_addr + k * kUmmaK * 2, 16, 1024);
                    const uint64_t bd = smem_desc_sw128(b_addr + k * kUmmaK * 2, 16, 1024);
                    umma_bf16_ss(tmem_base, ad, bd, idesc, (kb | k) ? 1u : 0u);
                }
                umma_commit(&ctl->empty[s]);
            }
            if (ok) umma_commit(&ctl->tmem_full);
        }
    } else {
        // ---------------- epilogue: tensor memory -> registers -> bf16 -> global ----------------
        const int quarter = warp & 3;                      // lanes this warp may read
        const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(&ctl->tmem_full, 0, abort_flag));
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        if (ok) {
            tc_fence_after_sync();
            const long long m = m0 + quarter * 32 + lane;
            const bool row_ok = m < g.p;
            __nv_bfloat16 *orow = out + (size_t)(row_ok ? m : 0) * g.cn + n0;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= g.cn) break;                 // warp-uniform
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        if (n0 + c0 + j < g.cn) {           // cn is a multiple of 8
                            float f[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                f[e] = __uint_as_float(v[j + e]);
                                if (bias) f[e] += __ldg(bias + n0 + c0 + j + e);
                            }
                            uint4 pk;
                            __nv_bfloat162 h;
                            h = __floats2bfloat162_rn(f[0], f[1]); pk.x = *(uint32_t *)&h;
                            h = __floats2bfloat162_rn(f[2], f[3]); pk.y = *(uint32_t *)&h;
                            h = __floats2bfloat162_rn(f[4], f[5]); pk.z = *(uint32_t *)&h;
                            h = __floats2bfloat162_rn(f[6], f[7]); pk.w = *(uint32_t *)&h;
                            *(uint4 *)(orow + c0 + j) = pk;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, BN);
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

bool umma_conv_eligible(const UmmaConvShape &s) {
    if (s.ca % kBK || s.cn % 8 || s.cn < 8) return false;
    if (s.lower_h < -128 || s.lower_h > 127 || s.lower_w < -128 || s.lower_w > 127) return false;
    if ((s.taps_h - 1) * s.dil_h > 255 || (s.taps_w - 1) * s.dil_w > 255) return false;
    if (s.stride_h > 8 || s.stride_w > 8) return false;
    if ((long long)s.taps_h * s.taps_w * s.ca > (1 << 24)) return false;
    return true;
}

template <int BN>
static cudaError_t launch_bn(const CUtensorMap &ta, const CUtensorMap &tw, ConvGemm g, const float *bias,
                             void *out, int *err, cudaStream_t st) {
    constexpr size_t stage = (size_t)kBM * kBK * 2 + (size_t)BN * kBK * 2;
    const int num_kb = g.taps_h * g.taps_w * (g.ca / kBK);
    int stages = (int)((96 * 1024) / stage);
    if (stages > num_kb) stages = num_kb;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 1) stages = 1;
    g.stages = stages;
    // Tensor memory has 512 columns per SM and every CTA takes BN of them: ask for enough shared
    // memory that no more than 512 / BN CTAs are resident, so an allocation never has to wait.
    size_t smem = stages * stage + 1024 + sizeof(ConvSmemCtl);
    const size_t floor_smem = (size_t)(228 * 1024) / (512 / BN + 1) + 1024;
    if (smem < floor_smem) smem = floor_smem;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(umma_conv_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             200 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    dim3 grid((unsigned)((g.p + kBM - 1) / kBM), (unsigned)((g.cn + BN - 1) / BN));
    umma_conv_kernel<BN><<<grid, kConvThreads, smem, st>>>(ta, tw, g, bias, (__nv_bfloat16 *)out, err);
    return cudaGetLastError();
}

cudaError_t launch_umma_conv(const UmmaConvShape &s, const void *act, const void *wmat, const float *bias,
                             void *out, cudaStream_t st) {
    ConvGemm g;
    g.ho = s.ho; g.wo = s.wo; g.cn = s.cn; g.ca = s.ca; g.taps_h = s.taps_h; g.taps_w = s.taps_w;
    g.lower_h = s.lower_h; g.lower_w = s.lower_w; g.stride_h = s.stride_h; g.stride_w = s.stride_w;
    g.dil_h = s.dil_h; g.dil_w = s.dil_w; g.p = (long long)s.n * s.ho * s.wo; g.stages = 1;
    // The bounding box of base pixels has ho x wo positions: upper = lower + (out-1) stride - (in-1).
    const int upper_h = s.lower_h + (s.ho - 1) * s.stride_h - (s.ha - 1);
    const int upper_w = s.lower_w + (s.wo - 1) * s.stride_w - (s.wa - 1);
    const long long tiles_m = (g.p + kBM - 1) / kBM;
    int bn = 64;
    if (s.cn > 64) {
        bn = (s.cn >= 256 && tiles_m * ((s.cn + 255) / 256) >= 148) ? 256 : 128;
        if (bn == 128 && tiles_m * ((s.cn + 127) / 128) < 148) bn = 64;
    }
    CUtensorMap ta, tw;
    if (!make_tmap_im2col_bf16(&ta, act, s.n, s.ha, s.wa, s.ca, s.lower_h, s.lower_w, upper_h, upper_w, s.stride_h,
                               s.stride_w, kBM, kBK))
        return cudaErrorInvalidValue;
    if (!make_tmap_matrix_bf16(&tw, wmat, s.cn, (long long)s.taps_h * s.taps_w * s.ca, bn, kBK))
        return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    if (bn == 64) return launch_bn<64>(ta, tw, g, bias, out, err, st);
    if (bn == 128) return launch_bn<128>(ta, tw, g, bias, out, err, st);
    return launch_bn<256>(ta, tw, g, bias, out, err, st);
}

}  // namespace convbn
