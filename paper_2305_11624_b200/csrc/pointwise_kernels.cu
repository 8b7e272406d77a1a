// Per-channel and elementwise kernels: omega' and b' formed from the current parameters at each call, per-channel
// sums, the parameter-gradient epilogue of Tune mode, and the Eval-mode BatchNorm passes.
#include <stdlib.h>

#include "kernels.h"

namespace convbn {

__device__ int g_error_word = 0;

namespace { thread_local int t_call_f16 = 0; }
void set_call_f16(int f16) { t_call_f16 = f16 ? 1 : 0; }
int call_f16() { return t_call_f16; }

int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    return dev;
}

int device_sm_count() {
    static int cache[kMaxDevices] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
    if (dev < 0 || dev >= kMaxDevices) dev = 0;
    if (!cache[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
        cache[dev] = v;
    }
    return cache[dev];
}

// The address is looked up once per device and cached, so launches make no runtime query
// (which also keeps them legal while a stream is being captured, after one warm-up call).
cudaError_t error_word_address(int **dev_ptr) {
    static int *cache[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaGetSymbolAddress((void **)dev_ptr, g_error_word);
    if (!cache[dev]) {
        int *p = nullptr;
        e = cudaGetSymbolAddress((void **)&p, g_error_word);
        if (e != cudaSuccess) return e;
        cache[dev] = p;
    }
    *dev_ptr = cache[dev];
    return cudaSuccess;
}

cudaError_t read_and_clear_error_word(int *host_value) {
    cudaError_t e = cudaMemcpyFromSymbol(host_value, g_error_word, sizeof(int));
    if (e != cudaSuccess) return e;
    const int zero = 0;
    return cudaMemcpyToSymbol(g_error_word, &zero, sizeof(int));
}

template <class F>
static cudaError_t by_type(int dtype, F f) {
    if (dtype == CONVBN_F32) return f((float *)0);
    if (dtype == CONVBN_BF16) return call_f16() ? f((__half *)0) : f((__nv_bfloat16 *)0);   // a half call runs as its bf16 twin
    return cudaErrorInvalidValue;
}

// ---- omega' = s omega, b' = (b - mu_hat) s + beta  (Sec. 3.3 definitions, used per step in Tune) ----
// One block row per output channel (blockIdx.y = co); the weight row keeps its memory order, so
// the kernel is layout-agnostic.
template <class T>
__global__ void __launch_bounds__(256) reparam_kernel(int c_out, int kdim, float eps,
                                                      const T *__restrict__ w,
                                                      const float *__restrict__ b,
                                                      const float *__restrict__ gamma,
                                                      const float *__restrict__ beta,
                                                      const float *__restrict__ mean,
                                                      const float *__restrict__ var,
                                                      float *__restrict__ vec3,
                                                      T *__restrict__ w_scaled,
                                                      float *__restrict__ b_fused) {
    const int co = blockIdx.y;
    const float r = 1.0f / sqrtf(var[co] + eps);
    const float s = gamma[co] * r;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const float bf = ((b ? b[co] : 0.f) - mean[co]) * s + beta[co];
        if (vec3) { vec3[co] = s; vec3[c_out + co] = bf; vec3[2 * c_out + co] = r; }
        if (b_fused) b_fused[co] = bf;
    }
    if (w_scaled) {
        const long long base = (long long)co * kdim;
        for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < kdim; k += gridDim.x * blockDim.x)
            w_scaled[base + k] = from_f32<T>(s * to_f32(w[base + k]));
    }
}

cudaError_t launch_reparam(const Problem &pb, int dtype, int layout, const void *w, const float *b,
                           const float *gamma, const float *beta, const float *mean,
                           const float *var, float *vec3, void *w_scaled, float *b_fused,
                           cudaStream_t st) {
    (void)layout;
    return by_type(dtype, [&](auto *tp) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        int gx = (pb.kdim + 255) / 256;
        if (gx > 8) gx = 8;
        if (!w_scaled) gx = 1;
        dim3 grid(gx, pb.c_out);
        reparam_kernel<T><<<grid, 256, 0, st>>>(pb.c_out, pb.kdim, pb.eps, (const T *)w, b, gamma,
                                                beta, mean, var, vec3, (T *)w_scaled, b_fused);
        return cudaGetLastError();
    });
}

template <class T>
__global__ void __launch_bounds__(256) rescale_weight_kernel(int kdim, const T *__restrict__ w,
                                                             const float *__restrict__ s_vec,
                                                             T *__restrict__ w_scaled, int reverse_row) {
    const int co = blockIdx.y;
    const float s = s_vec ? s_vec[co] : 1.f;
    const long long base = (long long)co * kdim;
    for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < kdim; k += gridDim.x * blockDim.x)
        w_scaled[base + (reverse_row ? kdim - 1 - k : k)] = from_f32<T>(s * to_f32(w[base + k]));
}

cudaError_t launch_rescale_weight(const Problem &pb, int dtype, const void *w, const float *vec3,
                                  void *w_scaled, cudaStream_t st, bool reverse_row) {
    return by_type(dtype, [&](auto *tp) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        int gx = (pb.kdim + 255) / 256;
        if (gx > 8) gx = 8;
        rescale_weight_kernel<T><<<dim3(gx, pb.c_out), 256, 0, st>>>(pb.kdim, (const T *)w, vec3, (T *)w_scaled,
                                                                     reverse_row ? 1 : 0);
        return cudaGetLastError();
    });
}

// omega' re-laid-out for the backward-data GEMM (dX = omega'_rot (*) dZ, Sec. 3.2.1): output channel
// becomes the contiguous (reduction) index and the taps are rotated by 180 degrees.
__global__ void __launch_bounds__(256) reparam_dgrad_kernel(int c_out, int c_in, int taps,
                                                            const __nv_bfloat16 *__restrict__ w,
                                                            const float *__restrict__ s_vec,
                                                            __nv_bfloat16 *__restrict__ w_t, int f16) {
    __shared__ float tile[32][33];
    pdl_wait();
    pdl_launch_dependents();
    const int tap = blockIdx.z, co0 = blockIdx.y * 32, ci0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int j = ty; j < 32; j += 8) {
        const int co = co0 + j, ci = ci0 + tx;
        if (co < c_out && ci < c_in)
            tile[j][tx] = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((long long)co * taps + tap) * c_in + ci, f16);
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
        const int ci = ci0 + j, co = co0 + tx;
        if (co < c_out && ci < c_in)
            reinterpret_cast<uint16_t *>(w_t)[((long long)ci * taps + (taps - 1 - tap)) * c_out + co] = pack1_h16(tile[tx][j], f16);
    }
}

__global__ void __launch_bounds__(256) reparam_dgrad_class_kernel(int c_out, int c_in, int kw, int tw, int r_max,
                                                                  int q_max, int step_h, int step_w, int ctaps,
                                                                  const __nv_bfloat16 *__restrict__ w,
                                                                  const float *__restrict__ s_vec,
                                                                  __nv_bfloat16 *__restrict__ w_t, int taps, int f16) {
    __shared__ float tile[32][33];
    pdl_wait();
    pdl_launch_dependents();
    const int ct = blockIdx.z, mh = ct / tw, mw = ct - mh * tw;
    const int tap = (r_max - step_h * mh) * kw + (q_max - step_w * mw);
    const int co0 = blockIdx.y * 32, ci0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int j = ty; j < 32; j += 8) {
        const int co = co0 + j, ci = ci0 + tx;
        if (co < c_out && ci < c_in)
            tile[j][tx] = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((long long)co * taps + tap) * c_in + ci, f16);
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
        const int ci = ci0 + j, co = co0 + tx;
        if (co < c_out && ci < c_in)
            reinterpret_cast<uint16_t *>(w_t)[((long long)ci * ctaps + ct) * c_out + co] = pack1_h16(tile[tx][j], f16);
    }
}

cudaError_t launch_reparam_dgrad_class(const Problem &pb, const void *w, const float *s_vec, void *w_t, int th,
                                       int tw, int r_max, int q_max, int step_h, int step_w, cudaStream_t st) {
    dim3 grid((pb.c_in + 31) / 32, (pb.c_out + 31) / 32, th * tw);
    static PerDevice carve;
    prefer_max_shared_once(reparam_dgrad_class_kernel, &carve);
    return launch_pdl(reparam_dgrad_class_kernel, grid, dim3(256), 0, st, pb.c_out, pb.c_in, pb.kw, tw, r_max, q_max,
                      step_h, step_w, th * tw, (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)w_t, pb.kh * pb.kw, call_f16());
}

// All residue classes of a strided backward pass in one launch: tap t of the kernel belongs to exactly
// one class; `where` gives, per tap, the element offset of its class matrix in w_t, the class's tap
// count and the tap's position in the class (count 0: the tap is not used).
__global__ void __launch_bounds__(256) reparam_dgrad_classes_kernel(int c_out, int c_in, ClassTapTable where,
                                                                    const __nv_bfloat16 *__restrict__ w,
                                                                    const float *__restrict__ s_vec,
                                                                    __nv_bfloat16 *__restrict__ w_t, int taps, int f16) {
    __shared__ float tile[32][33];
    pdl_wait();
    pdl_launch_dependents();
    const int tap = blockIdx.z, ctaps = where.count[tap], ct = where.pos[tap];
    if (ctaps == 0) return;
    __nv_bfloat16 *dst = w_t + where.offset[tap];
    const int co0 = blockIdx.y * 32, ci0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int j = ty; j < 32; j += 8) {
        const int co = co0 + j, ci = ci0 + tx;
        if (co < c_out && ci < c_in)
            tile[j][tx] = (s_vec ? s_vec[co] : 1.f) * load_h16(w + ((long long)co * taps + tap) * c_in + ci, f16);
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
        const int ci = ci0 + j, co = co0 + tx;
        if (co < c_out && ci < c_in) reinterpret_cast<uint16_t *>(dst)[((long long)ci * ctaps + ct) * c_out + co] = pack1_h16(tile[tx][j], f16);
    }
}

cudaError_t launch_reparam_dgrad_classes(const Problem &pb, const void *w, const float *s_vec, void *w_t,
                                         const ClassTapTable &where, cudaStream_t st) {
    dim3 grid((pb.c_in + 31) / 32, (pb.c_out + 31) / 32, pb.kh * pb.kw);
    static PerDevice carve;
    prefer_max_shared_once(reparam_dgrad_classes_kernel, &carve);
    return launch_pdl(reparam_dgrad_classes_kernel, grid, dim3(256), 0, st, pb.c_out, pb.c_in, where,
                      (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)w_t, pb.kh * pb.kw, call_f16());
}

cudaError_t launch_reparam_dgrad(const Problem &pb, const void *w, const float *s_vec, void *w_t,
                                 cudaStream_t st) {
    dim3 grid((pb.c_in + 31) / 32, (pb.c_out + 31) / 32, pb.kh * pb.kw);
    static PerDevice carve;
    prefer_max_shared_once(reparam_dgrad_kernel, &carve);
    return launch_pdl(reparam_dgrad_kernel, grid, dim3(256), 0, st, pb.c_out, pb.c_in, pb.kh * pb.kw,
                      (const __nv_bfloat16 *)w, s_vec, (__nv_bfloat16 *)w_t, call_f16());
}

// ---- per-channel partial sums over pixel slices (Appendix B) --------------------------------
template <class T, class L>
__global__ void __launch_bounds__(256) channel_sum_partial_kernel(int c_out, int h_out, int w_out,
                                                                  long long p, const T *__restrict__ t,
                                                                  float *__restrict__ part, int splits) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= c_out) return;
    const int split = blockIdx.y;
    const long long per = (p + splits - 1) / splits;
    const long long p0 = split * per, p1 = min(p, p0 + per);
    float acc = 0.f;
    if (L::id == CONVBN_NHWC) {
        for (long long q = p0; q < p1; ++q) acc += to_f32(t[q * c_out + c]);
    } else {
        const long long hw = (long long)h_out * w_out;
        for (long long q = p0; q < p1; ++q) {
            const long long n = q / hw, i = q % hw;
            acc += to_f32(t[(n * c_out + c) * hw + i]);
        }
    }
    part[(long long)split * c_out + c] = acc;
}

// NHWC, 16-bit elements (H: IEEE half, else bf16), C a multiple of 8: the tensor is a flat array of 16-byte
// vectors (8 channels); the block size is a multiple of C/8, so a thread always sees the same 8 channels.
// Per-thread sums are combined per channel in thread order (fixed), one partial row per block.
template <bool H>
__global__ void __launch_bounds__(256) channel_sum_nhwc8_kernel(int c_out, long long p, int pix_per_block,
                                                                const uint4 *__restrict__ t,
                                                                float *__restrict__ part) {
    __shared__ float red[256][9];
    const int v = c_out / 8;                       // vectors per pixel
    const long long vec0 = (long long)blockIdx.x * pix_per_block * v;
    long long vec1 = vec0 + (long long)pix_per_block * v;
    if (vec1 > p * v) vec1 = p * v;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (long long i = vec0 + threadIdx.x; i < vec1; i += blockDim.x) {
        const uint4 q = t[i];
        const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float lo, hi;
            unpack2_t<H>(u[e], lo, hi);
            acc[2 * e] += lo;
            acc[2 * e + 1] += hi;
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) red[threadIdx.x][e] = acc[e];
    __syncthreads();
    if ((int)threadIdx.x < c_out && (int)threadIdx.x < 256) {
        for (int c = threadIdx.x; c < c_out; c += blockDim.x) {
            const int g = c / 8, e = c % 8;
            float s = 0.f;
            for (int th = g; th < (int)blockDim.x; th += v) s += red[th][e];
            part[(long long)blockIdx.x * c_out + c] = s;
        }
    }
}

static bool channel_sum_fast(const Problem &pb, int dtype, int layout) {
    return dtype == CONVBN_BF16 && layout == CONVBN_NHWC && pb.c_out % 8 == 0 && pb.c_out / 8 <= 256;
}

int channel_sum_splits(const Problem &pb) {
    // shared by both kernels: about four blocks per SM, at least 64 pixels each
    long long want = 592;
    long long cap = (pb.p + 63) / 64;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    const long long per = (pb.p + want - 1) / want;
    return (int)((pb.p + per - 1) / per);
}

cudaError_t launch_channel_sum_partial(const Problem &pb, int dtype, int layout, const void *t,
                                       float *part, int splits, cudaStream_t st) {
    if (channel_sum_fast(pb, dtype, layout)) {
        const int v = pb.c_out / 8;
        const int block = (256 / v) * v;
        const long long per = (pb.p + splits - 1) / splits;
        if (call_f16()) channel_sum_nhwc8_kernel<true><<<splits, block, 0, st>>>(pb.c_out, pb.p, (int)per, (const uint4 *)t, part);
        else channel_sum_nhwc8_kernel<false><<<splits, block, 0, st>>>(pb.c_out, pb.p, (int)per, (const uint4 *)t, part);
        return cudaGetLastError();
    }
    const int threads = pb.c_out >= 256 ? 256 : ((pb.c_out + 31) / 32) * 32;
    dim3 grid((pb.c_out + threads - 1) / threads, splits);
    if (dtype == CONVBN_F32 && layout == CONVBN_NCHW)
        channel_sum_partial_kernel<float, NCHW><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, (const float *)t, part, splits);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC && call_f16())
        channel_sum_partial_kernel<__half, NHWC><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, (const __half *)t, part, splits);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC)
        channel_sum_partial_kernel<__nv_bfloat16, NHWC><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, (const __nv_bfloat16 *)t, part, splits);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

// ---- parameter-gradient epilogue (Table 2, Tune row: domega, db, dgamma, dbeta) -------------
// One block per output channel.  Partials are added in split order, then the row dot product
// sum_k domega'[co,k] omega[co,k] is reduced over the block in a fixed tree order.
template <class T>
__global__ void __launch_bounds__(256) wgrad_epilogue_kernel(int c_out, int kdim,
                                                             const float *__restrict__ partials, int splits,
                                                             const float *__restrict__ bsum_part, int bsplits,
                                                             const T *__restrict__ w,
                                                             const float *__restrict__ vec3,
                                                             const float *__restrict__ b,
                                                             const float *__restrict__ mean,
                                                             float *__restrict__ dw, float *__restrict__ db,
                                                             float *__restrict__ dgamma,
                                                             float *__restrict__ dbeta) {
    __shared__ float red[256];
    const int co = blockIdx.x;
    const long long rows = (long long)c_out * kdim;
    const float s = vec3 ? vec3[co] : 1.f;
    float dot = 0.f;
    for (int k = threadIdx.x; k < kdim; k += blockDim.x) {
        const long long o = (long long)co * kdim + k;
        float acc = 0.f;
        for (int sp = 0; sp < splits; ++sp) acc += partials[sp * rows + o];
        dw[o] = s * acc;
        if (vec3) dot = fmaf(acc, to_f32(w[o]), dot);
    }
    float bs = 0.f;
    if (bsum_part)
        for (int sp = threadIdx.x; sp < bsplits; sp += blockDim.x) bs += bsum_part[(long long)sp * c_out + co];
    // two fixed-order block reductions: dot, then bs
    red[threadIdx.x] = dot;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    const float dot_all = red[0];
    __syncthreads();
    red[threadIdx.x] = bs;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    if (threadIdx.x == 0) {
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

cudaError_t launch_wgrad_epilogue(const Problem &pb, int dtype, const float *partials, int splits,
                                  const float *bsum_part, int bsplits, const void *w,
                                  const float *vec3, const float *b, const float *mean, float *dw,
                                  float *db, float *dgamma, float *dbeta, cudaStream_t st) {
    return by_type(dtype, [&](auto *tp) {
        using T = typename std::remove_pointer<decltype(tp)>::type;
        wgrad_epilogue_kernel<T><<<pb.c_out, 256, 0, st>>>(pb.c_out, pb.kdim, partials, splits,
                                                           bsum_part, bsplits, (const T *)w, vec3, b,
                                                           mean, dw, db, dgamma, dbeta);
        return cudaGetLastError();
    });
}

// ---- Eval-mode BatchNorm, forward: z = s y + (beta - mean s)  (Sec. 3.1) ----------------------
template <class T, class L>
__global__ void __launch_bounds__(256) bn_eval_fwd_kernel(int c_out, long long hw, long long total,
                                                          const T *__restrict__ y,
                                                          const float *__restrict__ vec3,
                                                          T *__restrict__ z) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int c = L::id == CONVBN_NHWC ? (int)(i % c_out) : (int)((i / hw) % c_out);
        z[i] = from_f32<T>(fmaf(vec3[c], to_f32(y[i]), vec3[c_out + c]));
    }
}

// 16-bit NHWC (H: IEEE half, else bf16) with C a multiple of 8: 16-byte vectors; the block size is a multiple of
// C / 8, so a thread keeps its 8 channels (and their scale / shift in registers) over its grid-stride loop.
template <bool H>
__global__ void __launch_bounds__(256) bn_eval_fwd_nhwc8_kernel(int c_out, long long vecs, const uint4 *__restrict__ y,
                                                                const float *__restrict__ vec3,
                                                                uint4 *__restrict__ z) {
    const int v = c_out / 8, cv = threadIdx.x % v;
    float sc[8], sh[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { sc[e] = vec3[cv * 8 + e]; sh[e] = vec3[c_out + cv * 8 + e]; }
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < vecs;
         i += (long long)gridDim.x * blockDim.x) {
        const uint4 q = y[i];
        const uint32_t u[4] = {q.x, q.y, q.z, q.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float lo, hi;
            unpack2_t<H>(u[e], lo, hi);
            o[e] = pack2_t<H>(fmaf(sc[2 * e], lo, sh[2 * e]), fmaf(sc[2 * e + 1], hi, sh[2 * e + 1]));
        }
        z[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// dy = s dz and per-block partial sums of dz (y - mean) r and dz, one partial row per block
// (Table 2, Eval row); layout and block shape as above, lanes combined per channel in thread order.
template <bool H>
__global__ void __launch_bounds__(256) bn_eval_bwd_nhwc8_kernel(int c_out, long long p, int pix_per_block, float eps,
                                                                const uint4 *__restrict__ dz,
                                                                const uint4 *__restrict__ y,
                                                                const float *__restrict__ gamma,
                                                                const float *__restrict__ mean,
                                                                const float *__restrict__ var,
                                                                uint4 *__restrict__ dy, float *__restrict__ part_g,
                                                                float *__restrict__ part_b) {
    __shared__ float red[256][9];
    const int v = c_out / 8, cv = threadIdx.x % v;
    float s8[8], r8[8], m8[8], ag[8], ab[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int c = cv * 8 + e;
        r8[e] = 1.0f / sqrtf(var[c] + eps);
        s8[e] = gamma[c] * r8[e];
        m8[e] = mean[c];
        ag[e] = ab[e] = 0.f;
    }
    const long long vec0 = (long long)blockIdx.x * pix_per_block * v;
    long long vec1 = vec0 + (long long)pix_per_block * v;
    if (vec1 > p * v) vec1 = p * v;
    for (long long i = vec0 + threadIdx.x; i < vec1; i += blockDim.x) {
        const uint4 qd = dz[i], qy = y[i];
        const uint32_t ud[4] = {qd.x, qd.y, qd.z, qd.w}, uy[4] = {qy.x, qy.y, qy.z, qy.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float d0, d1, y0, y1;
            unpack2_t<H>(ud[e], d0, d1);
            unpack2_t<H>(uy[e], y0, y1);
            ag[2 * e] = fmaf(d0, (y0 - m8[2 * e]) * r8[2 * e], ag[2 * e]);
            ag[2 * e + 1] = fmaf(d1, (y1 - m8[2 * e + 1]) * r8[2 * e + 1], ag[2 * e + 1]);
            ab[2 * e] += d0;
            ab[2 * e + 1] += d1;
            o[e] = pack2_t<H>(s8[2 * e] * d0, s8[2 * e + 1] * d1);
        }
        dy[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int e = 0; e < 8; ++e) red[threadIdx.x][e] = pass ? ab[e] : ag[e];
        __syncthreads();
        for (int c = threadIdx.x; c < c_out; c += blockDim.x) {
            const int g = c / 8, e = c % 8;
            float sum = 0.f;
            for (int th = g; th < (int)blockDim.x; th += v) sum += red[th][e];
            (pass ? part_b : part_g)[(long long)blockIdx.x * c_out + c] = sum;
        }
        __syncthreads();
    }
}

cudaError_t launch_bn_eval_fwd(const Problem &pb, int dtype, int layout, const void *y,
                               const float *vec3, void *z, cudaStream_t st) {
    if (channel_sum_fast(pb, dtype, layout)) {
        const int v = pb.c_out / 8, block = (256 / v) * v;
        const long long vecs = pb.p * v;
        long long nb = (vecs + block - 1) / block;
        if (nb > device_sm_count() * 16) nb = device_sm_count() * 16;
        if (call_f16()) bn_eval_fwd_nhwc8_kernel<true><<<(int)nb, block, 0, st>>>(pb.c_out, vecs, (const uint4 *)y, vec3, (uint4 *)z);
        else bn_eval_fwd_nhwc8_kernel<false><<<(int)nb, block, 0, st>>>(pb.c_out, vecs, (const uint4 *)y, vec3, (uint4 *)z);
        return cudaGetLastError();
    }
    const long long total = pb.p * pb.c_out, hw = (long long)pb.h_out * pb.w_out;
    long long blocks = (total + 255) / 256;
    if (blocks > device_sm_count() * 32) blocks = device_sm_count() * 32;
    if (dtype == CONVBN_F32 && layout == CONVBN_NCHW)
        bn_eval_fwd_kernel<float, NCHW><<<(int)blocks, 256, 0, st>>>(pb.c_out, hw, total, (const float *)y, vec3, (float *)z);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC && call_f16())
        bn_eval_fwd_kernel<__half, NHWC><<<(int)blocks, 256, 0, st>>>(pb.c_out, hw, total, (const __half *)y, vec3, (__half *)z);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC)
        bn_eval_fwd_kernel<__nv_bfloat16, NHWC><<<(int)blocks, 256, 0, st>>>(
            pb.c_out, hw, total, (const __nv_bfloat16 *)y, vec3, (__nv_bfloat16 *)z);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

// ---- Eval-mode BatchNorm, backward (Table 2, Eval row) ---------------------------------------
// dy = s dz, and per pixel slice: part_g = sum dz (y - mean) r, part_b = sum dz.
template <class T, class L>
__global__ void __launch_bounds__(256) bn_eval_bwd_kernel(int c_out, int h_out, int w_out, long long p,
                                                          float eps, const T *__restrict__ dz,
                                                          const T *__restrict__ y,
                                                          const float *__restrict__ gamma,
                                                          const float *__restrict__ mean,
                                                          const float *__restrict__ var,
                                                          T *__restrict__ dy, float *__restrict__ part_g,
                                                          float *__restrict__ part_b, int splits) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= c_out) return;
    const int split = blockIdx.y;
    const long long per = (p + splits - 1) / splits;
    const long long p0 = split * per, p1 = min(p, p0 + per);
    const float r = 1.0f / sqrtf(var[c] + eps), s = gamma[c] * r, m = mean[c];
    const long long hw = (long long)h_out * w_out;
    float ag = 0.f, ab = 0.f;
    for (long long q = p0; q < p1; ++q) {
        const long long i = L::id == CONVBN_NHWC ? q * c_out + c : ((q / hw) * c_out + c) * hw + q % hw;
        const float d = to_f32(dz[i]);
        dy[i] = from_f32<T>(s * d);
        ag = fmaf(d, (to_f32(y[i]) - m) * r, ag);
        ab += d;
    }
    part_g[(long long)split * c_out + c] = ag;
    part_b[(long long)split * c_out + c] = ab;
}

cudaError_t launch_bn_eval_bwd(const Problem &pb, int dtype, int layout, const void *dz, const void *y,
                               const float *gamma, const float *mean, const float *var, void *dy,
                               float *part_g, float *part_b, int splits, cudaStream_t st) {
    if (channel_sum_fast(pb, dtype, layout)) {
        const int v = pb.c_out / 8, block = (256 / v) * v;
        const long long per = (pb.p + splits - 1) / splits;
        if (call_f16())
            bn_eval_bwd_nhwc8_kernel<true><<<splits, block, 0, st>>>(pb.c_out, pb.p, (int)per, pb.eps, (const uint4 *)dz,
                                                                     (const uint4 *)y, gamma, mean, var, (uint4 *)dy, part_g, part_b);
        else
            bn_eval_bwd_nhwc8_kernel<false><<<splits, block, 0, st>>>(pb.c_out, pb.p, (int)per, pb.eps, (const uint4 *)dz,
                                                                      (const uint4 *)y, gamma, mean, var, (uint4 *)dy, part_g, part_b);
        return cudaGetLastError();
    }
    const int threads = pb.c_out >= 256 ? 256 : ((pb.c_out + 31) / 32) * 32;
    dim3 grid((pb.c_out + threads - 1) / threads, splits);
    if (dtype == CONVBN_F32 && layout == CONVBN_NCHW)
        bn_eval_bwd_kernel<float, NCHW><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, pb.eps, (const float *)dz, (const float *)y, gamma, mean,
            var, (float *)dy, part_g, part_b, splits);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC && call_f16())
        bn_eval_bwd_kernel<__half, NHWC><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, pb.eps, (const __half *)dz, (const __half *)y, gamma, mean, var,
            (__half *)dy, part_g, part_b, splits);
    else if (dtype == CONVBN_BF16 && layout == CONVBN_NHWC)
        bn_eval_bwd_kernel<__nv_bfloat16, NHWC><<<grid, threads, 0, st>>>(
            pb.c_out, pb.h_out, pb.w_out, pb.p, pb.eps, (const __nv_bfloat16 *)dz,
            (const __nv_bfloat16 *)y, gamma, mean, var, (__nv_bfloat16 *)dy, part_g, part_b, splits);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

__global__ void bn_eval_finish_kernel(int c_out, float eps, const float *__restrict__ part_g,
                                      const float *__restrict__ part_b, int splits,
                                      const float *__restrict__ gamma, const float *__restrict__ var,
                                      float *__restrict__ db, float *__restrict__ dgamma,
                                      float *__restrict__ dbeta) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= c_out) return;
    float g = 0.f, bsum = 0.f;
    for (int sp = 0; sp < splits; ++sp) {
        g += part_g[(long long)sp * c_out + c];
        bsum += part_b[(long long)sp * c_out + c];
    }
    dgamma[c] = g;
    dbeta[c] = bsum;
    if (db) db[c] = gamma[c] / sqrtf(var[c] + eps) * bsum;
}

cudaError_t launch_bn_eval_finish(const Problem &pb, const float *part_g, const float *part_b,
                                  int splits, const float *gamma, const float *var, float *db,
                                  float *dgamma, float *dbeta, cudaStream_t st) {
    bn_eval_finish_kernel<<<(pb.c_out + 127) / 128, 128, 0, st>>>(pb.c_out, pb.eps, part_g, part_b, splits,
                                                                 gamma, var, db, dgamma, dbeta);
    return cudaGetLastError();
}

}  // namespace convbn
