// Elementwise glue between ConvBN blocks of a residual network: ReLU and the skip-connection add.  They are not
// part of the block (Sec. 3.1: the block is unaffected by the activation function or skip connection that
// follows it), but a whole-backbone replay needs them between the blocks, on the same stream and without
// allocations.  bf16, half or fp32 storage, fp32 arithmetic, 16-byte accesses, grid-stride loops.
#include "kernels.h"

namespace convbn {

namespace {

template <class T> struct Vec;
template <> struct Vec<__nv_bfloat16> { static constexpr int n = 8; };
template <> struct Vec<__half> { static constexpr int n = 8; };
template <> struct Vec<float> { static constexpr int n = 4; };

template <class T>
__device__ __forceinline__ void load_vec(const T *p, float (&f)[Vec<T>::n]) {
    const uint4 q = *(const uint4 *)p;
    if constexpr (Vec<T>::n == 8) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = unpack_h16((uint16_t)(w[i] & 0xFFFFu), sizeof(T) == 2 && !__is_same(T, __nv_bfloat16));
            f[2 * i + 1] = unpack_h16((uint16_t)(w[i] >> 16), sizeof(T) == 2 && !__is_same(T, __nv_bfloat16));
        }
    } else {
        f[0] = __uint_as_float(q.x); f[1] = __uint_as_float(q.y); f[2] = __uint_as_float(q.z); f[3] = __uint_as_float(q.w);
    }
}
template <class T>
__device__ __forceinline__ void store_vec(T *p, const float (&f)[Vec<T>::n]) {
    uint4 q;
    if constexpr (Vec<T>::n == 8) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = pack2_h16(f[2 * i], f[2 * i + 1], !__is_same(T, __nv_bfloat16));
        q = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
        q = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
    *(uint4 *)p = q;
}

// mode 0: out = max(a, 0)            mode 1: out = max(a + b, 0)
// mode 2: out = a where b > 0 else 0 (ReLU backward: a = gradient, b = ReLU output)      mode 3: out = a + b
template <class T, int MODE>
__global__ void __launch_bounds__(256) glue_kernel(const T *__restrict__ a, const T *__restrict__ b, T *__restrict__ out,
                                                   long long count) {
    constexpr int V = Vec<T>::n;
    pdl_wait();
    pdl_launch_dependents();
    const long long nvec = count / V;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        float x[V], y[V];
        load_vec(a + i * V, x);
        if (MODE != 0) load_vec(b + i * V, y);
#pragma unroll
        for (int k = 0; k < V; ++k) {
            if (MODE == 0) x[k] = fmaxf(x[k], 0.f);
            else if (MODE == 1) x[k] = fmaxf(x[k] + y[k], 0.f);
            else if (MODE == 2) x[k] = y[k] > 0.f ? x[k] : 0.f;
            else x[k] = x[k] + y[k];
        }
        store_vec(out + i * V, x);
    }
    // tail (count not a multiple of the vector width)
    if (blockIdx.x == 0 && threadIdx.x < (unsigned)(count - nvec * V)) {
        const long long i = nvec * V + threadIdx.x;
        const float x = to_f32(a[i]), y = MODE != 0 ? to_f32(b[i]) : 0.f;
        float r;
        if (MODE == 0) r = fmaxf(x, 0.f);
        else if (MODE == 1) r = fmaxf(x + y, 0.f);
        else if (MODE == 2) r = y > 0.f ? x : 0.f;
        else r = x + y;
        out[i] = from_f32<T>(r);
    }
}

template <class T, int MODE>
cudaError_t launch_glue_t(const void *a, const void *b, void *out, long long count, cudaStream_t st) {
    long long blocks = (count / Vec<T>::n + 255) / 256;
    const long long cap = (long long)device_sm_count() * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return launch_pdl(glue_kernel<T, MODE>, dim3((unsigned)blocks), dim3(256), 0, st, (const T *)a, (const T *)b, (T *)out, count);
}

}  // namespace

cudaError_t launch_glue(int mode, int dtype, const void *a, const void *b, void *out, long long count, cudaStream_t st) {
    if (dtype == CONVBN_F16) {
        switch (mode) {
            case 0: return launch_glue_t<__half, 0>(a, b, out, count, st);
            case 1: return launch_glue_t<__half, 1>(a, b, out, count, st);
            case 2: return launch_glue_t<__half, 2>(a, b, out, count, st);
            case 3: return launch_glue_t<__half, 3>(a, b, out, count, st);
            default: return cudaErrorInvalidValue;
        }
    }
    const bool bf = dtype == CONVBN_BF16;
    switch (mode) {
        case 0: return bf ? launch_glue_t<__nv_bfloat16, 0>(a, b, out, count, st) : launch_glue_t<float, 0>(a, b, out, count, st);
        case 1: return bf ? launch_glue_t<__nv_bfloat16, 1>(a, b, out, count, st) : launch_glue_t<float, 1>(a, b, out, count, st);
        case 2: return bf ? launch_glue_t<__nv_bfloat16, 2>(a, b, out, count, st) : launch_glue_t<float, 2>(a, b, out, count, st);
        case 3: return bf ? launch_glue_t<__nv_bfloat16, 3>(a, b, out, count, st) : launch_glue_t<float, 3>(a, b, out, count, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace convbn
