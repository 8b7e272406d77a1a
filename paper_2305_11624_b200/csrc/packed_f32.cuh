// Packed fp32 arithmetic (two values per register pair and instruction, sm_100) and the bf16 pair
// conversions that go with it.
#pragma once
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

}  // namespace convbn
