// Direct convolution kernels: one thread per output element, fp32 accumulation, any stride /
// padding / dilation / groups, both layouts and both storage types.  They serve the fp32 NCHW
// path and every shape the specialised kernels do not take.
#include "kernels.h"

namespace convbn {

// Z[n,co,ho,wo] = bias[co] + sum_{ci,r,q} W[co,ci,r,q] X[n, g cg + ci, ho sh - ph + r dh, wo sw - pw + q dw]
// (Sec. 3.1 forward; the weight is whatever the caller folded into it.)
template <class T, class L>
__global__ void __launch_bounds__(256) direct_fwd_kernel(Problem pb, const T *__restrict__ x,
                                                         const T *__restrict__ w,
                                                         const float *__restrict__ bias,
                                                         T *__restrict__ z) {
    const long long total = pb.p * pb.c_out;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int n, co, ho, wo;
        long long t = i;
        if (L::id == CONVBN_NCHW) {
            wo = t % pb.w_out; t /= pb.w_out; ho = t % pb.h_out; t /= pb.h_out;
            co = t % pb.c_out; n = (int)(t / pb.c_out);
        } else {
            co = t % pb.c_out; t /= pb.c_out; wo = t % pb.w_out; t /= pb.w_out;
            ho = t % pb.h_out; n = (int)(t / pb.h_out);
        }
        const int g = co / pb.cog;
        float acc = bias ? bias[co] : 0.f;
        for (int r = 0; r < pb.kh; ++r) {
            const int hi = ho * pb.stride_h - pb.pad_h + r * pb.dil_h;
            if (hi < 0 || hi >= pb.h_in) continue;
            for (int q = 0; q < pb.kw; ++q) {
                const int wi = wo * pb.stride_w - pb.pad_w + q * pb.dil_w;
                if (wi < 0 || wi >= pb.w_in) continue;
                for (int ci = 0; ci < pb.cg; ++ci) {
                    const float xv = to_f32(x[act_idx<L>(n, g * pb.cg + ci, hi, wi, pb.c_in, pb.h_in, pb.w_in)]);
                    const float wv = to_f32(w[w_idx<L>(co, ci, r, q, pb.cg, pb.kh, pb.kw)]);
                    acc = fmaf(xv, wv, acc);
                }
            }
        }
        z[i] = from_f32<T>(acc);
    }
}

// dX[n,c,h,w] = sum over (co in group, r, q) with ho sh - ph + r dh = h, wo sw - pw + q dw = w of
// W[co, c - g cg, r, q] dZ[n,co,ho,wo]      (Sec. 3.2.1: dX = omega_rot (*) dY, gathered per dX element)
template <class T, class L>
__global__ void __launch_bounds__(256) direct_dgrad_kernel(Problem pb, const T *__restrict__ dz,
                                                           const T *__restrict__ w,
                                                           T *__restrict__ dx) {
    const long long total = pb.pin * pb.c_in;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int n, c, h, wq;
        long long t = i;
        if (L::id == CONVBN_NCHW) {
            wq = t % pb.w_in; t /= pb.w_in; h = t % pb.h_in; t /= pb.h_in;
            c = t % pb.c_in; n = (int)(t / pb.c_in);
        } else {
            c = t % pb.c_in; t /= pb.c_in; wq = t % pb.w_in; t /= pb.w_in;
            h = t % pb.h_in; n = (int)(t / pb.h_in);
        }
        const int g = c / pb.cg, ci = c - g * pb.cg;
        float acc = 0.f;
        for (int r = 0; r < pb.kh; ++r) {
            const int hs = h + pb.pad_h - r * pb.dil_h;
            if (hs < 0 || hs % pb.stride_h) continue;
            const int ho = hs / pb.stride_h;
            if (ho >= pb.h_out) continue;
            for (int q = 0; q < pb.kw; ++q) {
                const int ws = wq + pb.pad_w - q * pb.dil_w;
                if (ws < 0 || ws % pb.stride_w) continue;
                const int wo = ws / pb.stride_w;
                if (wo >= pb.w_out) continue;
                for (int cc = 0; cc < pb.cog; ++cc) {
                    const int co = g * pb.cog + cc;
                    const float dv = to_f32(dz[act_idx<L>(n, co, ho, wo, pb.c_out, pb.h_out, pb.w_out)]);
                    const float wv = to_f32(w[w_idx<L>(co, ci, r, q, pb.cg, pb.kh, pb.kw)]);
                    acc = fmaf(dv, wv, acc);
                }
            }
        }
        dx[i] = from_f32<T>(acc);
    }
}

// partial[split][co][k] = sum over the split's pixels of dZ[p,co] X[p shifted by tap k]
// (Sec. 3.2.1: domega = dY (.) X, the reduction over N, H_out, W_out cut into slices).
template <class T, class L>
__global__ void __launch_bounds__(256) direct_wgrad_kernel(Problem pb, const T *__restrict__ dz,
                                                           const T *__restrict__ x,
                                                           float *__restrict__ partials, int splits) {
    const long long rows = (long long)pb.c_out * pb.kdim;
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const int split = blockIdx.y;
    const int co = (int)(i / pb.kdim), k = (int)(i % pb.kdim);
    int ci, r, q;
    w_row_decode<L>(k, pb.cg, pb.kh, pb.kw, ci, r, q);
    const int c = (co / pb.cog) * pb.cg + ci;
    const long long per = (pb.p + splits - 1) / splits;
    const long long p0 = split * per, p1 = min(pb.p, p0 + per);
    float acc = 0.f;
    if (p0 < p1) {
        int wo = (int)(p0 % pb.w_out);
        long long t = p0 / pb.w_out;
        int ho = (int)(t % pb.h_out), n = (int)(t / pb.h_out);
        for (long long p = p0; p < p1; ++p) {
            const int hi = ho * pb.stride_h - pb.pad_h + r * pb.dil_h;
            const int wi = wo * pb.stride_w - pb.pad_w + q * pb.dil_w;
            if (hi >= 0 && hi < pb.h_in && wi >= 0 && wi < pb.w_in) {
                const float dv = to_f32(dz[act_idx<L>(n, co, ho, wo, pb.c_out, pb.h_out, pb.w_out)]);
                const float xv = to_f32(x[act_idx<L>(n, c, hi, wi, pb.c_in, pb.h_in, pb.w_in)]);
                acc = fmaf(dv, xv, acc);
            }
            if (++wo == pb.w_out) { wo = 0; if (++ho == pb.h_out) { ho = 0; ++n; } }
        }
    }
    partials[(long long)split * rows + i] = acc;
}

template <class F>
static cudaError_t dispatch(int dtype, int layout, F f) {
    if (dtype == CONVBN_F32 && layout == CONVBN_NCHW) return f((float *)0, NCHW());
    if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC && call_f16()) return f((__half *)0, NHWC());   // a half call runs as its bf16 twin
    if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC) return f((__nv_bfloat16 *)0, NHWC());
    return cudaErrorInvalidValue;
}

static int grid_for(long long total) {
    long long b = (total + 255) / 256;
    const long long cap = (long long)device_sm_count() * 64;
    return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

cudaError_t launch_direct_fwd(const Problem &pb, int dtype, int layout, const void *x, const void *w,
                              const float *bias, void *z, cudaStream_t st) {
    return dispatch(dtype, layout, [&](auto *tp, auto L) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        direct_fwd_kernel<T, decltype(L)><<<grid_for(pb.p * pb.c_out), 256, 0, st>>>(
            pb, (const T *)x, (const T *)w, bias, (T *)z);
        return cudaGetLastError();
    });
}

cudaError_t launch_direct_dgrad(const Problem &pb, int dtype, int layout, const void *dz,
                                const void *w, void *dx, cudaStream_t st) {
    return dispatch(dtype, layout, [&](auto *tp, auto L) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        direct_dgrad_kernel<T, decltype(L)><<<grid_for(pb.pin * pb.c_in), 256, 0, st>>>(
            pb, (const T *)dz, (const T *)w, (T *)dx);
        return cudaGetLastError();
    });
}

int direct_wgrad_splits(const Problem &pb) {
    const long long rows = (long long)pb.c_out * pb.kdim;
    long long want = ((long long)device_sm_count() * 2048 * 2 + rows - 1) / rows;   // about two full waves of threads
    long long cap = pb.p / 32;                                // at least 32 pixels per slice
    if (cap < 1) cap = 1;
    if (want > cap) want = cap;
    if (want > 512) want = 512;
    if (want < 1) want = 1;
    return (int)want;
}

cudaError_t launch_direct_wgrad(const Problem &pb, int dtype, int layout, const void *dz,
                                const void *x, float *partials, int splits, cudaStream_t st) {
    return dispatch(dtype, layout, [&](auto *tp, auto L) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        const long long rows = (long long)pb.c_out * pb.kdim;
        dim3 grid((unsigned)((rows + 255) / 256), (unsigned)splits);
        direct_wgrad_kernel<T, decltype(L)><<<grid, 256, 0, st>>>(pb, (const T *)dz, (const T *)x,
                                                                  partials, splits);
        return cudaGetLastError();
    });
}

}  // namespace convbn
