// Depthwise 3x3 forward (and, with rotated taps, unit-stride backward data) as a streaming kernel fed by TMA.
//   Z[n,h,w,c] = b'[c] + sum_{r,q} omega'[c,r,q] X[n, h - p + r, w - p + q, c]      (Sec. 3.1 / 3.2.1 / 3.3)
// Depthwise convolution moves about one byte per 2 FLOP, so the kernel is organised around the memory
// stream: a producer warp issues one TMA box per input row ((strip width + KW - 1) pixels x C channels,
// out-of-image rows and columns filled with zeros by the copy engine) into a deep shared-memory ring, so
// that tens of KB per SM are in flight whatever the consumers do.  The consumer threads each own
// 4 channels x TW output columns, keep their KH x KW x 4 weights in registers, read each input row from
// shared memory once, widen it to fp32 once and add it into the KH output rows it reaches, whose
// accumulators rotate through KH register slots (row loop unrolled KH times, all indices static).  The
// arithmetic is packed fp32, two channels per FMA instruction.  A block walks down a band of `th` output
// rows of one column strip of one image, then takes its next (image, band, strip) item.
#include "kernels.h"
#include "packed_f32.cuh"
#include "sm100_ptx.cuh"

namespace convbn {

namespace {

using namespace ptx;

constexpr int kDwMaxStages = 32;

struct DwTmaCtl {
    uint64_t full[kDwMaxStages];
    uint64_t empty[kDwMaxStages];
    int abort_flag;
};

// Shared-memory accesses by 32-bit shared-space address (keeps the inner loop free of generic addressing).
__device__ __forceinline__ uint2 lds_u2(uint32_t addr) {
    uint2 r;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ bool try_wait_u32(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// 8-byte global store under a predicate (a predicated instruction: no branch, no reconvergence point)
__device__ __forceinline__ void stg_u2_if(void *ptr, uint32_t x, uint32_t y, bool on) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %3, 0;\n\t@p st.global.v2.b32 [%0], {%1, %2};\n\t}" ::"l"(ptr), "r"(x),
                 "r"(y), "r"((int)on)
                 : "memory");
}
// lane 0 of the warp arrives; a predicated instruction, so the warp does not branch
__device__ __forceinline__ void arrive_lane0(uint32_t bar, int lane) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.eq.s32 p, %1, 0;\n\t@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar),
        "r"(lane)
        : "memory");
}
// Slow part of a wait: polls for at most two seconds, and gives up early when another role has set the
// abort flag.  Returns false on give-up.
__device__ __forceinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (try_wait_u32(bar, parity)) return true;
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > 2000000000ull) return false;
        }
    }
}

struct DwTmaGeom {
    int n, c, h_in, w_in, h_out, w_out, pad_h, pad_w;
    int cols_t;        // consumer thread columns per block (each TW output columns wide)
    int strips;        // column strips per row
    int th, bands;     // output rows per band, bands per image
    int stages;        // ring depth
    int row_bytes;     // bytes of one TMA box
    int stage_stride;  // row_bytes rounded up to 128
    int consumer_warps;
};

template <int TW, int KH, int KW, bool H>
__global__ void __launch_bounds__(TW >= 4 ? 384 : 288, TW >= 4 ? 1 : 2) dw_tma_kernel(const __grid_constant__ CUtensorMap tx, DwTmaGeom g,
                                                        const __nv_bfloat16 *__restrict__ w,
                                                        const float *__restrict__ bias, const BnFold fold,
                                                        const float *__restrict__ scale, int reverse_taps,
                                                        uint2 *__restrict__ z, int *err) {
    constexpr int NX = TW + KW - 1;
    extern __shared__ uint8_t dw_smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dw_smem_raw) + 127) & ~(uintptr_t)127);
    DwTmaCtl *ctl = reinterpret_cast<DwTmaCtl *>(base);
    uint8_t *ring = base + ((sizeof(DwTmaCtl) + 127) / 128) * 128;
    volatile int *abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < g.stages; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], (uint32_t)g.consumer_warps);
        }
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const uint32_t items = (uint32_t)g.n * g.bands * g.strips;
    const int bwo = g.cols_t * TW;                             // output columns per strip
    if (warp == g.consumer_warps) {
        // ---- producer: one elected lane streams the input rows of every item of this block ----
        if (lane == 0) {
            prefetch_tensormap(&tx);
            uint32_t slot = 0, par = 0;                        // ring position of the next row
            bool ok = true;
            for (uint32_t it = blockIdx.x; it < items && ok; it += gridDim.x) {
                const int strip = (int)(it % (uint32_t)g.strips);
                const uint32_t t1 = it / (uint32_t)g.strips;
                const int band = (int)(t1 % (uint32_t)g.bands), img = (int)(t1 / (uint32_t)g.bands);
                const int rows = min(g.th, g.h_out - band * g.th), steps = rows + KH - 1;
                const int wi0 = strip * bwo - g.pad_w, hi0 = band * g.th - g.pad_h;
                for (int k = 0; k < steps; ++k) {
                    if (!mbar_wait_bounded(&ctl->empty[slot], par ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(&ctl->full[slot], (uint32_t)g.row_bytes);
                    tma_load_4d(ring + (size_t)slot * g.stage_stride, &tx, &ctl->full[slot], 0, wi0, hi0 + k, img);
                    if (++slot == (uint32_t)g.stages) { slot = 0; par ^= 1u; }
                }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
        return;
    }
    // ---- consumers ----
    const int v = g.c / 4;
    const int cv = (int)threadIdx.x % v, tc = (int)threadIdx.x / v;
    const bool active = tc < g.cols_t;
    f32x2 wr[KH * KW][2];
    f32x2 bv[2] = {0ull, 0ull};
    if (active) {
        // Per-channel factor of the taps: the BN fold formed here (forward, Sec. 3.3: s = gamma / sqrt(var +
        // eps), b' = (b - mu) s + beta; omega stays unrounded), or the saved s (backward data), or 1.
        float sc[4] = {1.f, 1.f, 1.f, 1.f}, bf[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int c = cv * 4 + e;
            if (fold.gamma) {
                const float r = 1.0f / sqrtf(fold.var[c] + fold.eps);
                sc[e] = fold.gamma[c] * r;
                bf[e] = ((fold.b ? fold.b[c] : 0.f) - fold.mean[c]) * sc[e] + fold.beta[c];
                if (blockIdx.x == 0 && tc == 0 && fold.vec3) {
                    fold.vec3[c] = sc[e]; fold.vec3[g.c + c] = bf[e]; fold.vec3[2 * g.c + c] = r;
                }
            } else {
                if (scale) sc[e] = scale[c];
                if (bias) bf[e] = bias[c];
            }
        }
#pragma unroll
        for (int tp = 0; tp < KH * KW; ++tp) {
            const int src = reverse_taps ? KH * KW - 1 - tp : tp;
            float f[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) f[e] = sc[e] * load_h16(w + (size_t)(cv * 4 + e) * (KH * KW) + src, H ? 1 : 0);
            wr[tp][0] = pair(f[0], f[1]);
            wr[tp][1] = pair(f[2], f[3]);
        }
        bv[0] = pair(bf[0], bf[1]);
        bv[1] = pair(bf[2], bf[3]);
    } else {
#pragma unroll
        for (int tp = 0; tp < KH * KW; ++tp) wr[tp][0] = wr[tp][1] = 0ull;
    }
    const uint32_t col_bytes = (uint32_t)g.c * 2;
    uint32_t col_addr[NX];                                     // this thread's columns in ring slot 0
#pragma unroll
    for (int j = 0; j < NX; ++j)
        col_addr[j] = smem_u32(ring) + (uint32_t)((active ? tc : 0) * TW + j) * col_bytes + (uint32_t)cv * 8;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    const uint32_t ring_bytes = (uint32_t)g.stages * g.stage_stride;
    uint32_t slot = 0, slot_off = 0, par = 0;                  // ring position of the next row
    const ptrdiff_t zpitch = (ptrdiff_t)g.w_out * v;
    bool ok = true;
    for (uint32_t it = blockIdx.x; it < items && ok; it += gridDim.x) {
        const int strip = (int)(it % (uint32_t)g.strips);
        const uint32_t t1 = it / (uint32_t)g.strips;
        const int band = (int)(t1 % (uint32_t)g.bands), img = (int)(t1 / (uint32_t)g.bands);
        const int rows = min(g.th, g.h_out - band * g.th);
        int steps = rows + KH - 1;
        const int wo0 = strip * bwo + tc * TW;
        // output row pointer, KH - 1 rows behind the input row being read
        uint2 *zr = z + ((ptrdiff_t)(img * g.h_out + band * g.th - (KH - 1)) * g.w_out + wo0) * v + cv;
        bool out_ok[TW];
#pragma unroll
        for (int j = 0; j < TW; ++j) out_ok[j] = active && wo0 + j < g.w_out;
        f32x2 acc[KH][TW][2];
#pragma unroll
        for (int sl = 0; sl < KH; ++sl)
#pragma unroll
            for (int j = 0; j < TW; ++j) acc[sl][j][0] = acc[sl][j][1] = 0ull;
        // step k brings input row (band start - pad_h + k), which is tap row r of output row k - r of the
        // band; output row o lives in slot o % KH, and k0 is a multiple of KH
        for (int k0 = 0; k0 < steps; k0 += KH) {
#pragma unroll
            for (int ph = 0; ph < KH; ++ph) {
                const int k = k0 + ph;
                if (k < steps) {
                    if (!try_wait_u32(full0 + slot * 8, par) && !wait_slow(full0 + slot * 8, par, abort_flag)) {
                        ok = false;
                        steps = 0;                             // leaves both loops
                    } else {
                        f32x2 xs[NX][2];
#pragma unroll
                        for (int j = 0; j < NX; ++j) {
                            const uint2 q = lds_u2(col_addr[j] + slot_off);
                            xs[j][0] = widen_t<H>(q.x);
                            xs[j][1] = widen_t<H>(q.y);
                        }
                        __syncwarp();
                        arrive_lane0(empty0 + slot * 8, lane);
                        ++slot;
                        slot_off += (uint32_t)g.stage_stride;
                        if (slot_off == ring_bytes) { slot = 0; slot_off = 0; par ^= 1u; }
                        // tap row 0 opens output row k in slot ph (from the bias); rows before the band's
                        // first or past its last only reach slots that are re-opened before, or never
                        // reach, a store
#pragma unroll
                        for (int r = 0; r < KH; ++r) {
                            const int sl = (ph - r + KH) % KH;
#pragma unroll
                            for (int q = 0; q < KW; ++q)
#pragma unroll
                                for (int j = 0; j < TW; ++j) {
                                    acc[sl][j][0] = fma2(xs[j + q][0], wr[r * KW + q][0],
                                                         (r == 0 && q == 0) ? bv[0] : acc[sl][j][0]);
                                    acc[sl][j][1] = fma2(xs[j + q][1], wr[r * KW + q][1],
                                                         (r == 0 && q == 0) ? bv[1] : acc[sl][j][1]);
                                }
                        }
                        {                                      // output row k - (KH - 1) is complete from k = KH - 1 on
                            const int sl = (ph + 1) % KH;
                            const bool row_done = k >= KH - 1;
#pragma unroll
                            for (int j = 0; j < TW; ++j)
                                stg_u2_if(zr + (ptrdiff_t)j * v, narrow_t<H>(acc[sl][j][0]), narrow_t<H>(acc[sl][j][1]), row_done && out_ok[j]);
                        }
                        zr += zpitch;
                    }
                }
            }
        }
    }
    if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
}

// ---- backward weight ---------------------------------------------------------------------------------
//   domega'[c,r,q] = sum_{n,h,w} dZ[n,h,w,c] X[n, h - p + r, w - p + q, c],   sum dZ[.,c]      (Sec. 3.2.1)
// The same row stream with two boxes per ring slot: the X row (with halo columns) and the dZ row of the
// same step.  X row k of a band meets dZ rows k, k-1, k-2 (tap rows 0, 1, 2), so every consumer keeps the
// last KH dZ rows of its columns in KH rotating register slots and its KH x KW x 4 sums (plus the sum of
// dZ) in registers across all the items of the block.  At the end the thread columns are added in
// column order through shared memory, and the block writes one partial row: part[block][c][KH KW + 1].
template <int TW, int KH, int KW, bool H>
__global__ void __launch_bounds__(TW >= 4 ? 384 : 288, TW >= 4 ? 1 : 2) dw_tma_wgrad_kernel(const __grid_constant__ CUtensorMap tx,
                                                              const __grid_constant__ CUtensorMap tdz, DwTmaGeom g,
                                                              float *__restrict__ part, int *err) {
    constexpr int NX = TW + KW - 1, NACC = KH * KW + 1;
    extern __shared__ uint8_t dw_smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dw_smem_raw) + 127) & ~(uintptr_t)127);
    DwTmaCtl *ctl = reinterpret_cast<DwTmaCtl *>(base);
    uint8_t *ring = base + ((sizeof(DwTmaCtl) + 127) / 128) * 128;
    volatile int *abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < g.stages; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], (uint32_t)g.consumer_warps);
        }
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const uint32_t items = (uint32_t)g.n * g.bands * g.strips;
    const int bwo = g.cols_t * TW;                             // dZ columns per strip
    const uint32_t x_bytes = (uint32_t)(bwo + KW - 1) * g.c * 2, dz_bytes = (uint32_t)bwo * g.c * 2;
    const uint32_t dz_off = (x_bytes + 127u) & ~127u;          // dZ row behind the X row in a slot
    const int v = g.c / 4;
    const int cv = (int)threadIdx.x % v, tc = (int)threadIdx.x / v;
    const bool active = warp < g.consumer_warps && tc < g.cols_t;
    f32x2 acc[NACC][2];
#pragma unroll
    for (int t = 0; t < NACC; ++t) acc[t][0] = acc[t][1] = 0ull;
    if (warp == g.consumer_warps) {
        // ---- producer ----
        if (lane == 0) {
            prefetch_tensormap(&tx);
            prefetch_tensormap(&tdz);
            uint32_t slot = 0, par = 0;
            bool ok = true;
            for (uint32_t it = blockIdx.x; it < items && ok; it += gridDim.x) {
                const int strip = (int)(it % (uint32_t)g.strips);
                const uint32_t t1 = it / (uint32_t)g.strips;
                const int band = (int)(t1 % (uint32_t)g.bands), img = (int)(t1 / (uint32_t)g.bands);
                const int rows = min(g.th, g.h_out - band * g.th), steps = rows + KH - 1;
                const int wo0 = strip * bwo, ho0 = band * g.th;
                for (int k = 0; k < steps; ++k) {
                    if (!mbar_wait_bounded(&ctl->empty[slot], par ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *dst = ring + (size_t)slot * g.stage_stride;
                    mbar_arrive_expect_tx(&ctl->full[slot], x_bytes + (k < rows ? dz_bytes : 0u));
                    tma_load_4d(dst, &tx, &ctl->full[slot], 0, wo0 - g.pad_w, ho0 - g.pad_h + k, img);
                    if (k < rows) tma_load_4d(dst + dz_off, &tdz, &ctl->full[slot], 0, wo0, ho0 + k, img);
                    if (++slot == (uint32_t)g.stages) { slot = 0; par ^= 1u; }
                }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
    } else {
        // ---- consumers ----
        const uint32_t col_bytes = (uint32_t)g.c * 2;
        uint32_t x_addr[NX], dz_addr[TW];
#pragma unroll
        for (int j = 0; j < NX; ++j)
            x_addr[j] = smem_u32(ring) + (uint32_t)((active ? tc : 0) * TW + j) * col_bytes + (uint32_t)cv * 8;
#pragma unroll
        for (int j = 0; j < TW; ++j)
            dz_addr[j] = smem_u32(ring) + dz_off + (uint32_t)((active ? tc : 0) * TW + j) * col_bytes + (uint32_t)cv * 8;
        const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
        const uint32_t ring_bytes = (uint32_t)g.stages * g.stage_stride;
        const f32x2 ones = pair(1.f, 1.f);
        uint32_t slot = 0, slot_off = 0, par = 0;
        bool ok = true;
        for (uint32_t it = blockIdx.x; it < items && ok; it += gridDim.x) {
            const uint32_t t1 = it / (uint32_t)g.strips;
            const int band = (int)(t1 % (uint32_t)g.bands);
            const int rows = min(g.th, g.h_out - band * g.th);
            int steps = rows + KH - 1;
            f32x2 dzw[KH][TW][2];                              // dZ row o of the band lives in slot o % KH
#pragma unroll
            for (int sl = 0; sl < KH; ++sl)
#pragma unroll
                for (int j = 0; j < TW; ++j) dzw[sl][j][0] = dzw[sl][j][1] = 0ull;
            for (int k0 = 0; k0 < steps; k0 += KH) {
#pragma unroll
                for (int ph = 0; ph < KH; ++ph) {
                    const int k = k0 + ph;
                    if (k < steps) {
                        if (!try_wait_u32(full0 + slot * 8, par) && !wait_slow(full0 + slot * 8, par, abort_flag)) {
                            ok = false;
                            steps = 0;                         // leaves both loops
                        } else {
                            f32x2 xs[NX][2];
#pragma unroll
                            for (int j = 0; j < NX; ++j) {
                                const uint2 q = lds_u2(x_addr[j] + slot_off);
                                xs[j][0] = widen_t<H>(q.x);
                                xs[j][1] = widen_t<H>(q.y);
                            }
                            if (k < rows) {                    // same for the whole block
#pragma unroll
                                for (int j = 0; j < TW; ++j) {
                                    const uint2 q = lds_u2(dz_addr[j] + slot_off);
                                    dzw[ph][j][0] = widen_t<H>(q.x);
                                    dzw[ph][j][1] = widen_t<H>(q.y);
                                    acc[KH * KW][0] = fma2(dzw[ph][j][0], ones, acc[KH * KW][0]);
                                    acc[KH * KW][1] = fma2(dzw[ph][j][1], ones, acc[KH * KW][1]);
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < TW; ++j) dzw[ph][j][0] = dzw[ph][j][1] = 0ull;
                            }
                            __syncwarp();
                            arrive_lane0(empty0 + slot * 8, lane);
                            ++slot;
                            slot_off += (uint32_t)g.stage_stride;
                            if (slot_off == ring_bytes) { slot = 0; slot_off = 0; par ^= 1u; }
                            // X row k is tap row r of dZ row k - r (slot (ph - r) mod KH; zero outside the band)
#pragma unroll
                            for (int r = 0; r < KH; ++r) {
                                const int sl = (ph - r + KH) % KH;
#pragma unroll
                                for (int q = 0; q < KW; ++q)
#pragma unroll
                                    for (int j = 0; j < TW; ++j) {
                                        acc[r * KW + q][0] = fma2(dzw[sl][j][0], xs[j + q][0], acc[r * KW + q][0]);
                                        acc[r * KW + q][1] = fma2(dzw[sl][j][1], xs[j + q][1], acc[r * KW + q][1]);
                                    }
                            }
                        }
                    }
                }
            }
        }
        if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    }
    // ---- add the thread columns (in column order) and write the block's partial row ----
    __syncthreads();                                           // every row has been consumed: the ring is free
    float *red = reinterpret_cast<float *>(ring);              // [cols_t][C / 4][NACC][4]
    if (active) {
        float *mine = red + ((size_t)tc * v + cv) * (NACC * 4);
#pragma unroll
        for (int t = 0; t < NACC; ++t) {
            float a, b, c2, d;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(acc[t][0]));
            asm("mov.b64 {%0, %1}, %2;" : "=f"(c2), "=f"(d) : "l"(acc[t][1]));
            *reinterpret_cast<float4 *>(mine + t * 4) = make_float4(a, b, c2, d);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < g.c * NACC; i += blockDim.x) {
        const int c = i / NACC, t = i - c * NACC;
        float sum = 0.f;
        for (int col = 0; col < g.cols_t; ++col) sum += red[((size_t)col * v + c / 4) * (NACC * 4) + t * 4 + (c & 3)];
        part[(size_t)blockIdx.x * g.c * NACC + i] = sum;
    }
}

// Adds the block partials in block order and forms the parameter gradients (Table 2, Tune row):
//   domega = s domega', dbeta = sum dZ, db = s dbeta, dgamma = r (sum_k domega' omega + dbeta (b - mu_hat)).
// vec3 == NULL: domega = domega', db = sum dZ.  One block per channel; warp t sums tap t (warp KH KW: dZ).
template <int TAPS>
__global__ void __launch_bounds__(32 * (TAPS + 1)) dw_wgrad_finish_kernel(int c_total, int nparts,
                                                                           const float *__restrict__ part,
                                                                           const __nv_bfloat16 *__restrict__ w,
                                                                           const float *__restrict__ vec3,
                                                                           const float *__restrict__ b,
                                                                           const float *__restrict__ mean,
                                                                           float *__restrict__ dw, float *__restrict__ db,
                                                                           float *__restrict__ dgamma,
                                                                           float *__restrict__ dbeta, int f16) {
    __shared__ float tot[TAPS + 1];
    const int c = blockIdx.x, t = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float sum = 0.f;
    for (int p = lane; p < nparts; p += 32) sum += part[((size_t)p * c_total + c) * (TAPS + 1) + t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    if (lane == 0) tot[t] = sum;
    __syncthreads();
    if (threadIdx.x < TAPS) dw[(size_t)c * TAPS + threadIdx.x] = (vec3 ? vec3[c] : 1.f) * tot[threadIdx.x];
    if (threadIdx.x == 0) {
        const float dsum = tot[TAPS];
        if (vec3) {
            float dot = 0.f;
            for (int k = 0; k < TAPS; ++k) dot = fmaf(tot[k], load_h16(w + (size_t)c * TAPS + k, f16), dot);
            const float s = vec3[c], r = vec3[2 * c_total + c];
            dbeta[c] = dsum;
            if (db) db[c] = s * dsum;
            dgamma[c] = r * (dot + dsum * ((b ? b[c] : 0.f) - mean[c]));
        } else if (db) {
            db[c] = dsum;
        }
    }
}

}  // namespace

bool dw_tma_eligible(const Problem &pb) {
    return pb.groups == pb.c_in && pb.c_in == pb.c_out && pb.c_in % 8 == 0 && pb.c_in <= 256 && pb.kh == 3 &&
           pb.kw == 3 && pb.stride_h == 1 && pb.stride_w == 1 && pb.dil_h == 1 && pb.dil_w == 1 && pb.pad_h >= 0 &&
           pb.pad_w >= 0 && pb.pad_h <= 2 && pb.pad_w <= 2 && pb.w_out >= 8 && pb.p * pb.c_out < (1LL << 31) &&
           pb.pin * pb.c_in < (1LL << 31);
}

// Strip width, ring depth, band height and grid for a stream of `bytes_per_col_row` bytes per output
// column and row (X box plus, for the backward-weight kernel, the dZ box).
static cudaError_t dw_tma_geometry(const Problem &pb, int tw, int kh, int kw, bool with_dz, DwTmaGeom *out,
                                   unsigned *grid) {
    // consumer threads (the producer warp comes on top): two blocks of 256 per SM, or one block of 352 when a
    // thread owns four columns (its accumulators need the registers of a whole SM's worth of fewer threads)
    const int max_consumers = tw >= 4 ? 352 : 256;
    const size_t ring_budget = tw >= 4 ? 192 * 1024 : 96 * 1024;
    DwTmaGeom g{};
    g.n = pb.n; g.c = pb.c_in; g.h_in = pb.h_in; g.w_in = pb.w_in; g.h_out = pb.h_out; g.w_out = pb.w_out;
    g.pad_h = pb.pad_h; g.pad_w = pb.pad_w;
    const int v = pb.c_in / 4;
    const int tcols = (pb.w_out + tw - 1) / tw;                // thread columns in a row
    int cols_max = max_consumers / v;
    if (cols_max < 1) cols_max = 1;
    if (cols_max > 254 / tw) cols_max = 254 / tw;              // box width (cols tw + kw - 1) <= 256
    if (cols_max > tcols) cols_max = tcols;
    g.strips = (tcols + cols_max - 1) / cols_max;
    g.cols_t = (tcols + g.strips - 1) / g.strips;
    g.consumer_warps = (g.cols_t * v + 31) / 32;
    g.row_bytes = (g.cols_t * tw + kw - 1) * pb.c_in * 2;
    g.stage_stride = (g.row_bytes + 127) / 128 * 128;
    if (with_dz) g.stage_stride += (g.cols_t * tw * pb.c_in * 2 + 127) / 128 * 128;
    g.stages = (int)(ring_budget / g.stage_stride);
    if (g.stages > kDwMaxStages) g.stages = kDwMaxStages;
    if (g.stages < 4) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const long long resident = (tw >= 4 ? 1LL : 2LL) * sms;
    // band height: the one that minimises (items per block, rounded up) x (input rows per item)
    long long best = -1;
    g.th = pb.h_out;
    for (int th = 4; th <= pb.h_out; ++th) {
        const long long bands = (pb.h_out + th - 1) / th;
        const long long per_block = ((long long)pb.n * bands * g.strips + resident - 1) / resident;
        const long long cost = per_block * (th + kh - 1);
        if (best < 0 || cost < best) { best = cost; g.th = th; }
    }
    g.bands = (pb.h_out + g.th - 1) / g.th;
    const long long items = (long long)pb.n * g.bands * g.strips;
    *grid = (unsigned)(items < resident ? items : resident);
    *out = g;
    return cudaSuccess;
}

static bool dw_tma_map(CUtensorMap *tm, const void *base, int n, int h, int w, int c, int box_w) {
    const unsigned long long dims[4] = {(unsigned long long)c, (unsigned long long)w, (unsigned long long)h,
                                        (unsigned long long)n};
    const unsigned long long str[4] = {0, (unsigned long long)c * 2, (unsigned long long)w * c * 2,
                                       (unsigned long long)h * w * c * 2};
    const unsigned int box[4] = {(unsigned)c, (unsigned)box_w, 1, 1};
    return make_tmap_tiled_bf16_linear(tm, base, 4, dims, str, box);
}

static size_t dw_tma_smem(const DwTmaGeom &g) {
    return 128 + ((sizeof(DwTmaCtl) + 127) / 128) * 128 + (size_t)g.stages * g.stage_stride;
}

// fold != NULL: Tune forward from the raw weights and BN parameters (writes the saved vectors too);
// scale != NULL: taps multiplied by scale[c]; reverse_taps: taps read in reverse order (the rotated
// kernel of the backward-data pass on the mirrored problem).
cudaError_t launch_dw_tma(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                          cudaStream_t st, const BnFold *fold, const float *scale, bool reverse_taps) {
    constexpr int TW = 4, KH = 3, KW = 3;
    DwTmaGeom g;
    unsigned grid = 0;
    cudaError_t e = dw_tma_geometry(pb, TW, KH, KW, false, &g, &grid);
    if (e != cudaSuccess) return e;
    CUtensorMap tx;
    if (!dw_tma_map(&tx, x, pb.n, pb.h_in, pb.w_in, pb.c_in, g.cols_t * TW + KW - 1)) return cudaErrorInvalidValue;
    int *err = nullptr;
    if ((e = error_word_address(&err)) != cudaSuccess) return e;
    static PerDevice attr, attr_h;        // (one flag per instantiation)
    const BnFold none{nullptr, nullptr, nullptr, nullptr, nullptr, 0.f, nullptr};
    if (call_f16()) {
        if ((e = max_dynamic_smem_once(dw_tma_kernel<TW, KH, KW, true>, 210 * 1024, &attr_h)) != cudaSuccess) return e;
        dw_tma_kernel<TW, KH, KW, true><<<grid, (g.consumer_warps + 1) * 32, dw_tma_smem(g), st>>>(
            tx, g, (const __nv_bfloat16 *)w, bias, fold ? *fold : none, scale, reverse_taps ? 1 : 0, (uint2 *)z, err);
        return cudaGetLastError();
    }
    if ((e = max_dynamic_smem_once(dw_tma_kernel<TW, KH, KW, false>, 210 * 1024, &attr)) != cudaSuccess) return e;
    dw_tma_kernel<TW, KH, KW, false><<<grid, (g.consumer_warps + 1) * 32, dw_tma_smem(g), st>>>(
        tx, g, (const __nv_bfloat16 *)w, bias, fold ? *fold : none, scale, reverse_taps ? 1 : 0, (uint2 *)z, err);
    return cudaGetLastError();
}

// Partial rows the backward-weight kernel writes: one per block, [C][KH KW + 1] floats each.
size_t dw_tma_wgrad_partial_bytes(const Problem &pb) {
    DwTmaGeom g;
    unsigned grid = 0;
    if (dw_tma_geometry(pb, 4, 3, 3, true, &g, &grid) != cudaSuccess) return 0;
    return (size_t)grid * pb.c_in * 10 * sizeof(float);
}

cudaError_t launch_dw_tma_wgrad(const Problem &pb, const void *dz, const void *x, float *part, int *nparts,
                                cudaStream_t st) {
    constexpr int TW = 4, KH = 3, KW = 3;
    DwTmaGeom g;
    unsigned grid = 0;
    cudaError_t e = dw_tma_geometry(pb, TW, KH, KW, true, &g, &grid);
    if (e != cudaSuccess) return e;
    CUtensorMap tx, tdz;
    if (!dw_tma_map(&tx, x, pb.n, pb.h_in, pb.w_in, pb.c_in, g.cols_t * TW + KW - 1)) return cudaErrorInvalidValue;
    if (!dw_tma_map(&tdz, dz, pb.n, pb.h_out, pb.w_out, pb.c_in, g.cols_t * TW)) return cudaErrorInvalidValue;
    int *err = nullptr;
    if ((e = error_word_address(&err)) != cudaSuccess) return e;
    static PerDevice attr, attr_h;
    *nparts = (int)grid;
    if (call_f16()) {
        if ((e = max_dynamic_smem_once(dw_tma_wgrad_kernel<TW, KH, KW, true>, 210 * 1024, &attr_h)) != cudaSuccess) return e;
        dw_tma_wgrad_kernel<TW, KH, KW, true><<<grid, (g.consumer_warps + 1) * 32, dw_tma_smem(g), st>>>(tx, tdz, g, part, err);
        return cudaGetLastError();
    }
    if ((e = max_dynamic_smem_once(dw_tma_wgrad_kernel<TW, KH, KW, false>, 210 * 1024, &attr)) != cudaSuccess) return e;
    dw_tma_wgrad_kernel<TW, KH, KW, false><<<grid, (g.consumer_warps + 1) * 32, dw_tma_smem(g), st>>>(tx, tdz, g, part, err);
    return cudaGetLastError();
}

cudaError_t launch_dw_wgrad_finish(const Problem &pb, const float *part, int nparts, const void *w, const float *vec3,
                                   const float *b, const float *mean, float *dw, float *db, float *dgamma,
                                   float *dbeta, cudaStream_t st) {
    dw_wgrad_finish_kernel<9><<<pb.c_in, 32 * 10, 0, st>>>(pb.c_in, nparts, part, (const __nv_bfloat16 *)w, vec3, b, mean,
                                                         dw, db, dgamma, dbeta, call_f16());
    return cudaGetLastError();
}

}  // namespace convbn
