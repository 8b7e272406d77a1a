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
__device__ __forceinline__ void arrive_u32(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Out-of-line part of a wait: polls for at most two seconds, and gives up early when another role has
// set the abort flag.  Returns false on give-up.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
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

template <int TW, int KH, int KW>
__global__ void __launch_bounds__(288, 2) dw_tma_kernel(const __grid_constant__ CUtensorMap tx, DwTmaGeom g,
                                                        const __nv_bfloat16 *__restrict__ w,
                                                        const float *__restrict__ bias, uint2 *__restrict__ z,
                                                        int *err) {
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
#pragma unroll
        for (int tp = 0; tp < KH * KW; ++tp) {
            float f[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) f[e] = __bfloat162float(w[(size_t)(cv * 4 + e) * (KH * KW) + tp]);
            wr[tp][0] = pair(f[0], f[1]);
            wr[tp][1] = pair(f[2], f[3]);
        }
        if (bias) {
            const float4 f = *reinterpret_cast<const float4 *>(bias + cv * 4);
            bv[0] = pair(f.x, f.y);
            bv[1] = pair(f.z, f.w);
        }
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
                            xs[j][0] = widen(q.x);
                            xs[j][1] = widen(q.y);
                        }
                        __syncwarp();
                        if (lane == 0) arrive_u32(empty0 + slot * 8);
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
                        if (k >= KH - 1) {                     // output row k - (KH - 1) is complete
                            const int sl = (ph + 1) % KH;
#pragma unroll
                            for (int j = 0; j < TW; ++j)
                                if (out_ok[j]) zr[(ptrdiff_t)j * v] = make_uint2(narrow(acc[sl][j][0]), narrow(acc[sl][j][1]));
                        }
                        zr += zpitch;
                    }
                }
            }
        }
    }
    if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
}

}  // namespace

bool dw_tma_eligible(const Problem &pb) {
    return pb.groups == pb.c_in && pb.c_in == pb.c_out && pb.c_in % 8 == 0 && pb.c_in <= 256 && pb.kh == 3 &&
           pb.kw == 3 && pb.stride_h == 1 && pb.stride_w == 1 && pb.dil_h == 1 && pb.dil_w == 1 && pb.pad_h >= 0 &&
           pb.pad_w >= 0 && pb.pad_h <= 2 && pb.pad_w <= 2 && pb.w_out >= 8 && pb.p * pb.c_out < (1LL << 31) &&
           pb.pin * pb.c_in < (1LL << 31);
}

cudaError_t launch_dw_tma(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                          cudaStream_t st) {
    constexpr int TW = 2, KH = 3, KW = 3;
    DwTmaGeom g{};
    g.n = pb.n; g.c = pb.c_in; g.h_in = pb.h_in; g.w_in = pb.w_in; g.h_out = pb.h_out; g.w_out = pb.w_out;
    g.pad_h = pb.pad_h; g.pad_w = pb.pad_w;
    const int v = pb.c_in / 4;
    const int tcols = (pb.w_out + TW - 1) / TW;               // thread columns in a row
    int cols_max = 256 / v;                                    // at most 256 consumer threads
    if (cols_max < 1) cols_max = 1;
    if (cols_max > 254 / TW) cols_max = 254 / TW;              // box width (cols TW + KW - 1) <= 256
    if (cols_max > tcols) cols_max = tcols;
    g.strips = (tcols + cols_max - 1) / cols_max;
    g.cols_t = (tcols + g.strips - 1) / g.strips;
    g.consumer_warps = (g.cols_t * v + 31) / 32;
    g.row_bytes = (g.cols_t * TW + KW - 1) * pb.c_in * 2;
    g.stage_stride = (g.row_bytes + 127) / 128 * 128;
    g.stages = (int)((96 * 1024) / g.stage_stride);
    if (g.stages > kDwMaxStages) g.stages = kDwMaxStages;
    if (g.stages < 4) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const long long resident = 2LL * sms;
    // band height: the one that minimises (items per block, rounded up) x (input rows per item)
    long long best = -1;
    g.th = pb.h_out;
    for (int th = 4; th <= pb.h_out; ++th) {
        const long long bands = (pb.h_out + th - 1) / th;
        const long long per_block = ((long long)pb.n * bands * g.strips + resident - 1) / resident;
        const long long cost = per_block * (th + KH - 1);
        if (best < 0 || cost < best) { best = cost; g.th = th; }
    }
    if (pb.h_out < 4) g.th = pb.h_out;
    g.bands = (pb.h_out + g.th - 1) / g.th;
    const long long items = (long long)pb.n * g.bands * g.strips;
    const unsigned grid = (unsigned)(items < resident ? items : resident);

    CUtensorMap tx;
    const unsigned long long dims[4] = {(unsigned long long)pb.c_in, (unsigned long long)pb.w_in,
                                        (unsigned long long)pb.h_in, (unsigned long long)pb.n};
    const unsigned long long str[4] = {0, (unsigned long long)pb.c_in * 2, (unsigned long long)pb.w_in * pb.c_in * 2,
                                       (unsigned long long)pb.h_in * pb.w_in * pb.c_in * 2};
    const unsigned int box[4] = {(unsigned)pb.c_in, (unsigned)(g.cols_t * TW + KW - 1), 1, 1};
    if (!make_tmap_tiled_bf16_linear(&tx, x, 4, dims, str, box)) return cudaErrorInvalidValue;
    int *err = nullptr;
    if ((e = error_word_address(&err)) != cudaSuccess) return e;
    const size_t smem = 128 + ((sizeof(DwTmaCtl) + 127) / 128) * 128 + (size_t)g.stages * g.stage_stride;
    static bool attr = false;
    if (!attr) {
        e = cudaFuncSetAttribute(dw_tma_kernel<TW, KH, KW>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    dw_tma_kernel<TW, KH, KW><<<grid, (g.consumer_warps + 1) * 32, smem, st>>>(tx, g, (const __nv_bfloat16 *)w, bias,
                                                                              (uint2 *)z, err);
    return cudaGetLastError();
}

}  // namespace convbn
