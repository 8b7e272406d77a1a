// Pointwise kernels of the Tune-mode TransposedConv-BN block.  The transposed convolution itself runs on the
// convolution kernels of the layer it transposes (its forward pass is that layer's backward data and vice versa);
// what differs is the axis the per-channel scale lives on: the weights are [C_in][taps][C_out/G] (NHWC) or
// [C_in][C_out/G][taps] (NCHW) and s belongs to the OUTPUT channel, the inner axis.
#include "kernels.h"

namespace convbn {
namespace {

// output channel of weight element idx
__device__ __forceinline__ int tconv_channel(long long idx, int taps, int cig, int cog, bool nhwc) {
    int j, ci;
    if (nhwc) {
        j = (int)(idx % cog);
        ci = (int)(idx / ((long long)cog * taps));
    } else {
        j = (int)((idx / taps) % cog);
        ci = (int)(idx / ((long long)cog * taps));
    }
    return (ci / cig) * cog + j;
}

// vec3 = [s | b' | r]  (Sec. 3.3 definitions)
__global__ void tconv_vec3_kernel(int c_out, float eps, const float *__restrict__ b, const float *__restrict__ gamma,
                                  const float *__restrict__ beta, const float *__restrict__ mean,
                                  const float *__restrict__ var, float *__restrict__ vec3) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= c_out) return;
    const float r = 1.0f / sqrtf(var[c] + eps), s = gamma[c] * r;
    vec3[c] = s;
    vec3[c_out + c] = ((b ? b[c] : 0.0f) - mean[c]) * s + beta[c];
    vec3[2 * c_out + c] = r;
}

template <class T>
__global__ void __launch_bounds__(256) tconv_rescale_kernel(long long count, int taps, int cig, int cog, bool nhwc,
                                                            const T *__restrict__ w, const float *__restrict__ s,
                                                            T *__restrict__ w_out) {
    pdl_wait();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
        w_out[i] = from_f32<T>(to_f32(w[i]) * s[tconv_channel(i, taps, cig, cog, nhwc)]);
}

// z += b' per channel, in place
template <class T>
__global__ void __launch_bounds__(256) tconv_bias_kernel(long long count, int c, long long hw, bool nhwc,
                                                         const float *__restrict__ bias, T *__restrict__ z) {
    pdl_wait();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        const int ch = nhwc ? (int)(i % c) : (int)((i / hw) % c);
        z[i] = from_f32<T>(to_f32(z[i]) + bias[ch]);
    }
}

// One block per 32 output channels, 8 row slices per channel.  domega = s domega', dbeta = sum dZ, db = s dbeta,
// dgamma = r (sum over C_in/G and taps of domega' omega + dbeta (b - mu_hat))          (Table 2, Tune row)
template <class T>
__global__ void __launch_bounds__(256) tconv_param_epilogue_kernel(int c_out, int taps, int cig, int cog, bool nhwc,
                                                                   const float *__restrict__ dwp, const T *__restrict__ w,
                                                                   const float *__restrict__ vec3, const float *__restrict__ b,
                                                                   const float *__restrict__ mean,
                                                                   const float *__restrict__ bsum, int bsplits,
                                                                   float *__restrict__ dw, float *__restrict__ db,
                                                                   float *__restrict__ dgamma, float *__restrict__ dbeta) {
    pdl_wait();
    __shared__ float part[8][33];
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int co = blockIdx.x * 32 + lane;
    float dot = 0.0f;
    if (co < c_out) {
        const int g = co / cog, j = co - g * cog;
        const float s = vec3[co];
        const int rows = cig * taps;                   // (ci, tap) pairs of this channel's group
        for (int rr = slice; rr < rows; rr += 8) {
            const int ci = g * cig + rr / taps, tap = rr - (rr / taps) * taps;
            const long long idx = nhwc ? ((long long)ci * taps + tap) * cog + j : ((long long)ci * cog + j) * taps + tap;
            const float v = dwp[idx];
            dot = fmaf(v, to_f32(w[idx]), dot);
            dw[idx] = s * v;
        }
    }
    part[slice][lane] = dot;
    __syncthreads();
    if (slice == 0 && co < c_out) {
        float d = 0.0f, sum = 0.0f;
        for (int q = 0; q < 8; ++q) d += part[q][lane];
        for (int q = 0; q < bsplits; ++q) sum += bsum[(long long)q * c_out + co];
        const float s = vec3[co], r = vec3[2 * c_out + co];
        dbeta[co] = sum;
        if (db) db[co] = s * sum;
        dgamma[co] = r * (d + sum * ((b ? b[co] : 0.0f) - mean[co]));
    }
}

int grid_for(long long count) {
    long long blocks = (count + 255) / 256;
    const long long cap = (long long)device_sm_count() * 16;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace

cudaError_t launch_tconv_vec3(int c_out, float eps, const float *b, const float *gamma, const float *beta,
                              const float *mean, const float *var, float *vec3, cudaStream_t st) {
    tconv_vec3_kernel<<<(c_out + 127) / 128, 128, 0, st>>>(c_out, eps, b, gamma, beta, mean, var, vec3);
    return cudaGetLastError();
}

cudaError_t launch_tconv_rescale(int dtype, bool nhwc, long long count, int taps, int cig, int cog, const void *w,
                                 const float *s, void *w_out, cudaStream_t st) {
    if (dtype == CONVBN_BF16 && call_f16())     // a half call runs as its bf16 twin
        return launch_pdl(tconv_rescale_kernel<__half>, dim3(grid_for(count)), dim3(256), 0, st, count, taps, cig, cog, nhwc,
                          (const __half *)w, s, (__half *)w_out);
    if (dtype == CONVBN_BF16)
        return launch_pdl(tconv_rescale_kernel<__nv_bfloat16>, dim3(grid_for(count)), dim3(256), 0, st, count, taps, cig, cog,
                          nhwc, (const __nv_bfloat16 *)w, s, (__nv_bfloat16 *)w_out);
    return launch_pdl(tconv_rescale_kernel<float>, dim3(grid_for(count)), dim3(256), 0, st, count, taps, cig, cog, nhwc,
                      (const float *)w, s, (float *)w_out);
}

cudaError_t launch_tconv_bias(int dtype, bool nhwc, long long count, int c, long long hw, const float *bias, void *z,
                              cudaStream_t st) {
    if (dtype == CONVBN_BF16 && call_f16())
        return launch_pdl(tconv_bias_kernel<__half>, dim3(grid_for(count)), dim3(256), 0, st, count, c, hw, nhwc, bias, (__half *)z);
    if (dtype == CONVBN_BF16)
        return launch_pdl(tconv_bias_kernel<__nv_bfloat16>, dim3(grid_for(count)), dim3(256), 0, st, count, c, hw, nhwc, bias,
                          (__nv_bfloat16 *)z);
    return launch_pdl(tconv_bias_kernel<float>, dim3(grid_for(count)), dim3(256), 0, st, count, c, hw, nhwc, bias, (float *)z);
}

cudaError_t launch_tconv_param_epilogue(int dtype, bool nhwc, int c_out, int taps, int cig, int cog, const float *dwp,
                                        const void *w, const float *vec3, const float *b, const float *mean,
                                        const float *bsum, int bsplits, float *dw, float *db, float *dgamma,
                                        float *dbeta, cudaStream_t st) {
    const dim3 grid((c_out + 31) / 32);
    if (dtype == CONVBN_BF16 && call_f16())
        return launch_pdl(tconv_param_epilogue_kernel<__half>, grid, dim3(256), 0, st, c_out, taps, cig, cog, nhwc, dwp,
                          (const __half *)w, vec3, b, mean, bsum, bsplits, dw, db, dgamma, dbeta);
    if (dtype == CONVBN_BF16)
        return launch_pdl(tconv_param_epilogue_kernel<__nv_bfloat16>, grid, dim3(256), 0, st, c_out, taps, cig, cog, nhwc, dwp,
                          (const __nv_bfloat16 *)w, vec3, b, mean, bsum, bsplits, dw, db, dgamma, dbeta);
    return launch_pdl(tconv_param_epilogue_kernel<float>, grid, dim3(256), 0, st, c_out, taps, cig, cog, nhwc, dwp,
                      (const float *)w, vec3, b, mean, bsum, bsplits, dw, db, dgamma, dbeta);
}

}  // namespace convbn
