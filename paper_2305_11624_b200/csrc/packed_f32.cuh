// Packed fp32 arithmetic (two values per register pair and instruction, sm_100) and the bf16 pair
// conversions that go with it.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cstdint>

namespace convbn {

typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pair(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// two bf16 in one word -> two fp32
__device__ __forceinline__ f32x2 widen(uint32_t u) { return pair(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u)); }
// two fp32 -> two bf16 in one word (round to nearest even)
__device__ __forceinline__ uint32_t narrow(f32x2 p) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}
// The same for either 16-bit storage type, fixed at compile time (H: IEEE half, else bf16) or at run time.
template <bool H>
__device__ __forceinline__ f32x2 widen_t(uint32_t u) {
    if constexpr (H) { const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&u)); return pair(f.x, f.y); }
    else return widen(u);
}
template <bool H>
__device__ __forceinline__ uint32_t narrow_t(f32x2 p) {
    if constexpr (H) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
        const __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t *>(&h);
    } else return narrow(p);
}
__device__ __forceinline__ f32x2 widen_h16(uint32_t u, int f16) { return f16 ? widen_t<true>(u) : widen(u); }
__device__ __forceinline__ uint32_t narrow_h16(f32x2 p, int f16) { return f16 ? narrow_t<true>(p) : narrow(p); }

}  // namespace convbn
