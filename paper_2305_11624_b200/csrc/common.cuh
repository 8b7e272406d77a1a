// Shared device/host declarations of the ConvBN library: the kernel-side problem record,
// tensor index helpers for the two memory layouts, storage-type conversion and error plumbing.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "../../include/convbn.h"

namespace convbn {

// Problem sizes as the kernels see them (derived once on the host from convbn_desc).
struct Problem {
    int n, c_in, h_in, w_in, c_out, kh, kw;
    int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, groups;
    int h_out, w_out;
    int cg;        // input channels per group
    int cog;       // output channels per group
    int kdim;      // cg * kh * kw : length of one weight row
    long long p;   // n * h_out * w_out : output pixels
    long long pin; // n * h_in * w_in : input pixels
    float eps;
};

// Layout tags (match convbn_layout).
struct NCHW { static constexpr int id = CONVBN_NCHW; };
struct NHWC { static constexpr int id = CONVBN_NHWC; };

template <class L>
__host__ __device__ __forceinline__ long long act_idx(int n, int c, int h, int w, int C, int H, int W) {
    if (L::id == CONVBN_NCHW) return (((long long)n * C + c) * H + h) * W + w;
    return (((long long)n * H + h) * W + w) * C + c;
}

// Weight element (co, ci, r, q) of a [C_out][Cg][kh][kw] (NCHW) or [C_out][kh][kw][Cg] (NHWC) tensor.
template <class L>
__host__ __device__ __forceinline__ long long w_idx(int co, int ci, int r, int q, int cg, int kh, int kw) {
    if (L::id == CONVBN_NCHW) return (((long long)co * cg + ci) * kh + r) * kw + q;
    return (((long long)co * kh + r) * kw + q) * cg + ci;
}

// Position k within a weight row -> (ci, r, q) for the layout's row order.
template <class L>
__host__ __device__ __forceinline__ void w_row_decode(int k, int cg, int kh, int kw, int &ci, int &r, int &q) {
    if (L::id == CONVBN_NCHW) { q = k % kw; int t = k / kw; r = t % kh; ci = t / kh; }
    else { ci = k % cg; int t = k / cg; q = t % kw; r = t / kw; }
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
template <class T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// ---- the two 16-bit storage types ---------------------------------------------------------------------
// The tensor-core kernels move 16-bit elements without looking at them (TMA, shared memory, MMA operands);
// only four things depend on whether those bits are bf16 or IEEE half: the operand-format field of the MMA
// instruction descriptor, the conversion of results, the conversion of weights that are rescaled on the way,
// and the constant 1.  Those kernels carry an `f16` flag (0: bf16, 1: half) instead of a second instantiation.
// Kernels that do arithmetic on every element (depthwise, grouped warp-level MMAs, direct, element-wise) are
// templates on the type or take the same flag.
__device__ __forceinline__ uint32_t pack2_h16(float a, float b, int f16) {
    if (f16) { const __half2 h = __floats2half2_rn(a, b); return *reinterpret_cast<const uint32_t *>(&h); }
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&h);
}
// The same with the type fixed at compile time, for the epilogue loops (one uniform branch per tile picks the loop).
template <bool F16>
__device__ __forceinline__ uint32_t pack2_t(float a, float b) {
    if constexpr (F16) { const __half2 h = __floats2half2_rn(a, b); return *reinterpret_cast<const uint32_t *>(&h); }
    else { const __nv_bfloat162 h = __floats2bfloat162_rn(a, b); return *reinterpret_cast<const uint32_t *>(&h); }
}
template <bool F16>
__device__ __forceinline__ void unpack2_t(uint32_t bits, float &lo, float &hi) {
    if constexpr (F16) { const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&bits)); lo = f.x; hi = f.y; }
    else { lo = __uint_as_float(bits << 16); hi = __uint_as_float(bits & 0xFFFF0000u); }
}
__device__ __forceinline__ uint16_t pack1_h16(float a, int f16) {
    if (f16) { const __half h = __float2half_rn(a); return *reinterpret_cast<const uint16_t *>(&h); }
    const __nv_bfloat16 h = __float2bfloat16_rn(a);
    return *reinterpret_cast<const uint16_t *>(&h);
}
__device__ __forceinline__ float unpack_h16(uint16_t bits, int f16) {
    if (f16) return __half2float(*reinterpret_cast<const __half *>(&bits));
    return __uint_as_float((uint32_t)bits << 16);
}
__device__ __forceinline__ float load_h16(const void *p, int f16) { return unpack_h16(*reinterpret_cast<const uint16_t *>(p), f16); }
__host__ __device__ constexpr uint32_t one_h16(int f16) { return f16 ? 0x3C00u : 0x3F80u; }
// The storage type of the call in progress on this host thread (set by the entry points, read by the
// launchers when they fill their kernels' parameter records).
void set_call_f16(int f16);
int call_f16();

// Device error word: kernels that give up on a bounded wait OR a non-zero code into it.  The word
// lives in one translation unit; kernels elsewhere get its device address as an argument.
enum : int { ERRW_TIMEOUT = 1 };
cudaError_t error_word_address(int **dev_ptr);          // address on the current device
cudaError_t read_and_clear_error_word(int *host_value); // synchronous

// ---- programmatic dependent launch -------------------------------------------------------------
// Kernels launched through launch_pdl may start while the kernel before them in the stream is still
// running: their set-up (barriers, tensor memory, descriptor prefetch) then overlaps its tail.  They
// call pdl_wait() before their first access to global memory, which returns only once every earlier
// kernel has completed and flushed; launched the plain way, pdl_wait() returns at once.
// Invariant for kernels that own tensor memory: pdl_launch_dependents() comes only after the CTA's
// tcgen05.alloc has completed (after the block barrier that follows it).  A dependent CTA that became
// resident on the same SM earlier could take the columns first and then sit in its pdl_wait() for this
// grid, while this CTA's allocation blocks behind it.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- per-device facts ------------------------------------------------------------------------------
// Function attributes, the SM count and symbol addresses belong to a device, not to the process, so
// every cache below is keyed by the ordinal of the CURRENT device.
constexpr int kMaxDevices = 64;
int current_device_slot();      // ordinal of the current device in [0, kMaxDevices), 0 when none can be queried
int device_sm_count();          // SMs of the current device; 148 (B200) when no device is present (host-only sizing)
struct PerDevice { bool done[kMaxDevices] = {}; };


template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Ask for the largest shared-memory carve-out for a kernel, once per device.  The tensor-core kernels
// need it; the small kernels launched between them ask for the same split so that the SMs are not
// re-partitioned (which drains them) at every kernel boundary of a training step.
template <class K>
inline void prefer_max_shared_once(K kernel, PerDevice *flag) {
    bool &done = flag->done[current_device_slot()];
    if (done) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    done = true;
}
// Raise a kernel's dynamic shared-memory limit, once per device.
template <class K>
inline cudaError_t max_dynamic_smem_once(K kernel, int bytes, PerDevice *flag) {
    bool &done = flag->done[current_device_slot()];
    if (done) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done = true;
    return e;
}

// Hook for timing builds: a build that force-includes a header defining CONVBN_TRACE_POINT records a
// timestamp per CTA at the marked places; in the library it compiles to nothing.
#ifndef CONVBN_TRACE_POINT
#define CONVBN_TRACE_POINT(id) ((void)0)
#define CONVBN_TRACE_T0() ((void)0)            // start of a wait ...
#define CONVBN_TRACE_ACC(id) ((void)0)         // ... whose duration is added to slot id
#endif

static inline int ceil_div_i(long long a, long long b) { return (int)((a + b - 1) / b); }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace convbn
