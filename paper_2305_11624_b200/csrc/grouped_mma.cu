// Grouped convolution with 8 channels per group (C_in/G = C_out/G = 8), bf16 NHWC, unit stride and dilation:
//   Z[p, 8g + o] = b'[8g + o] + sum_{tap, ci} omega'[8g + o][tap][ci] X[p + tap, 8g + ci]     (Sec. 3.1 / 3.3)
// and, with rotated and transposed weights, the backward-data pass (Sec. 3.2.1).
// One group is a GEMM with N = 8 and K = 8 per tap (about 36 FLOP per byte moved): far too narrow for a
// 128-row tcgen05 tile, whose block-diagonal emulation spends 8x the MMA work and was bound by it, but an
// exact fit for the warp-level m16n8k16 MMA: 16 pixels x (2 taps x 8 input channels) x 8 output channels.
// The kernel is organised around the memory stream.  Work item = (image, band of R output rows, 64-channel
// chunk); a producer warp brings the item's input patch ((R + kh - 1) rows x (W + kw - 1) columns x 64
// channels, zero fill outside the image) into a ring of shared-memory stages with one TMA box (128-byte
// swizzle).  Compute warp w owns group w of the chunk: its A fragments are ldmatrix loads of [pixel][8
// channels] rows at the tap's shifted start address (virtual pixels, row pitch W + kw - 1: the outputs of
// the halo columns are computed and dropped), which the swizzle makes bank-conflict free; its B fragments
// (the group's 8 x 8 weights per tap) sit in registers for the whole item; results go straight to global
// memory as bf16 pairs.
#include "kernels.h"
#include "mma_sync.cuh"
#include "sm100_ptx.cuh"

namespace convbn {

namespace {

using namespace ptx;

constexpr int kGMaxStages = 8;
constexpr int kGMaxKSteps = 5;       // up to 10 taps (3 x 3), two per k-step; the loops over them are unrolled
constexpr int kGThreads = 288;       // 8 compute warps + the producer warp
constexpr int kGTiles = 4;           // 16-pixel MMA tiles a warp works on at a time

struct GroupedCtl {
    uint64_t full[kGMaxStages], empty[kGMaxStages];
    int abort_flag;
};

struct GroupedGeom {
    int n, ho, wo, c, kh, kw, lower_h, lower_w;
    int R, Wt, rows_in, tiles_h;
    int stages;
    uint32_t patch_bytes;      // bytes one TMA box writes
    uint32_t stage_stride;     // allocation per stage (multiple of 1024, includes the read-ahead tail)
};

template <bool H>            // H: IEEE-half storage, else bf16
__global__ void __launch_bounds__(kGThreads) grouped8_conv_kernel(const __grid_constant__ CUtensorMap tm_act,
                                                                 const GroupedGeom g,
                                                                 const __nv_bfloat16 *__restrict__ w,
                                                                 const float *__restrict__ bias,
                                                                 __nv_bfloat16 *__restrict__ out, int *err) {
    extern __shared__ uint8_t grouped_smem_raw[];
    uint8_t *ring = (uint8_t *)(((uintptr_t)grouped_smem_raw + 1023) & ~(uintptr_t)1023);
    GroupedCtl *ctl = (GroupedCtl *)(ring + (size_t)g.stages * g.stage_stride);
    volatile int *abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int taps = g.kh * g.kw, ksteps = (taps + 1) / 2, chunks = g.c / 64;
    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 8); }
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) { CONVBN_TRACE_POINT(0); }
    const uint32_t items = (uint32_t)g.n * g.tiles_h * chunks;   // chunk fastest: the chunks of a patch run together
    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&tm_act);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (uint32_t it = blockIdx.x; it < items; it += gridDim.x) {
                const int cc = (int)(it % (uint32_t)chunks);
                const uint32_t t1 = it / (uint32_t)chunks;
                const int h0 = (int)(t1 % (uint32_t)g.tiles_h) * g.R, img = (int)(t1 / (uint32_t)g.tiles_h);
                if (!mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                mbar_arrive_expect_tx(&ctl->full[s], g.patch_bytes);
                tma_load_4d(ring + (size_t)s * g.stage_stride, &tm_act, &ctl->full[s], cc * 64, g.lower_w,
                            h0 + g.lower_h, img);
                if (++s == (uint32_t)g.stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
        return;
    }
    // ---- compute warps: warp = group inside the 64-channel chunk ----
    const int gr = lane >> 2, t = lane & 3;
    // ldmatrix.x4: lanes 0-7 address the rows of matrix 0 (pixels 0-7, first tap), 8-15 matrix 1 (pixels
    // 8-15, first tap), 16-23 matrix 2 (pixels 0-7, second tap), 24-31 matrix 3 (pixels 8-15, second tap)
    const int lm_pix = (lane & 7) + ((lane >> 3) & 1) * 8, lm_tap = lane >> 4;
    const int npix = g.R * g.Wt;                               // virtual pixels of a full band
    uint32_t s = 0, ph = 0;
    bool ok = true;
    for (uint32_t it = blockIdx.x; it < items && ok; it += gridDim.x) {
        const int cc = (int)(it % (uint32_t)chunks);
        const uint32_t t1 = it / (uint32_t)chunks;
        const int h0 = (int)(t1 % (uint32_t)g.tiles_h) * g.R, img = (int)(t1 / (uint32_t)g.tiles_h);
        const int ch0 = cc * 64 + warp * 8;                    // first channel of this warp's group
        // B fragments: k = 8 (tap in the step) + ci, n = output channel gr; lane holds ci = 2t, 2t + 1
        uint32_t bf[kGMaxKSteps][2];
        const __nv_bfloat16 *wrow = w + ((size_t)(ch0 + gr) * taps) * 8 + 2 * t;
#pragma unroll
        for (int ks = 0; ks < kGMaxKSteps; ++ks) {
            bf[ks][0] = 2 * ks < taps ? *reinterpret_cast<const uint32_t *>(wrow + (size_t)(2 * ks) * 8) : 0u;
            bf[ks][1] = 2 * ks + 1 < taps ? *reinterpret_cast<const uint32_t *>(wrow + (size_t)(2 * ks + 1) * 8) : 0u;
        }
        const float b0 = bias ? bias[ch0 + 2 * t] : 0.f, b1 = bias ? bias[ch0 + 2 * t + 1] : 0.f;
        // this lane's ldmatrix row of k-step ks, relative to the tile start: its pixel plus the shift of its tap
        int vrow[kGMaxKSteps];
        {
            int r = 0, q = 0;                                  // tap 2 ks
#pragma unroll
            for (int ks = 0; ks < kGMaxKSteps; ++ks) {
                int r1 = r, q1 = q + 1;                        // tap 2 ks + 1
                if (q1 == g.kw) { q1 = 0; ++r1; }
                const bool second = lm_tap && 2 * ks + 1 < taps;   // an absent second tap re-reads the first (weights 0)
                vrow[ks] = lm_pix + (second ? r1 * g.Wt + q1 : r * g.Wt + q);
                r = r1; q = q1 + 1;
                if (q >= g.kw) { q -= g.kw; ++r; }
            }
        }
        const int rows_here = min(g.R, g.ho - h0);
        __nv_bfloat16 *obase = out + ((size_t)((size_t)img * g.ho + h0) * g.wo) * g.c + ch0 + 2 * t;
        const int wrap_elems = (g.wo - g.Wt) * g.c;            // output offset of (row + 1, column - Wt)
        if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
        if (threadIdx.x == 0) { if (it == blockIdx.x) CONVBN_TRACE_POINT(1); CONVBN_TRACE_POINT(3); }
        const uint32_t patch = smem_u32(ring + (size_t)s * g.stage_stride);
        // four 16-pixel tiles at a time: their MMA chains are independent, so the loads of one overlap
        // the arithmetic of the others
        for (int v0 = 0; v0 < npix; v0 += 16 * kGTiles) {
            float acc[kGTiles][4];
#pragma unroll
            for (int u = 0; u < kGTiles; ++u) { acc[u][0] = b0; acc[u][1] = b1; acc[u][2] = b0; acc[u][3] = b1; }
#pragma unroll
            for (int ks = 0; ks < kGMaxKSteps; ++ks) {
                if (ks >= ksteps) break;                       // the same for every lane
                const int v = v0 + vrow[ks];
                // tiles are 16 rows = 2048 bytes apart, which leaves the swizzle term unchanged
                const uint32_t addr = patch + (uint32_t)v * 128u + (uint32_t)((warp ^ (v & 7)) << 4);
                uint32_t a[kGTiles][4];
#pragma unroll
                for (int u = 0; u < kGTiles; ++u) ldmatrix_x4(a[u][0], a[u][1], a[u][2], a[u][3], addr + (uint32_t)u * 2048u);
#pragma unroll
                for (int u = 0; u < kGTiles; ++u) mma_16x8x16_t<H>(acc[u], a[u][0], a[u][1], a[u][2], a[u][3], bf[ks][0], bf[ks][1]);
            }
            // rows gr and gr + 8 of tile u are virtual pixels v0 + 16 u + gr (+ 8): walk them, 8 pixels a step
            int ti = (v0 + gr) / g.Wt, tj = (v0 + gr) - ti * g.Wt;
            ptrdiff_t off = ((ptrdiff_t)ti * g.wo + tj) * g.c;
#pragma unroll
            for (int u = 0; u < kGTiles; ++u)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (ti < rows_here && tj < g.wo)
                        *reinterpret_cast<uint32_t *>(obase + off) = pack2_t<H>(acc[u][2 * half], acc[u][2 * half + 1]);
                    tj += 8;
                    off += 8 * g.c;
                    if (tj >= g.Wt) { tj -= g.Wt; ++ti; off += wrap_elems; }
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[s]);
        if (threadIdx.x == 0) { if (it == blockIdx.x) CONVBN_TRACE_POINT(2); CONVBN_TRACE_POINT(4); }
        if (++s == (uint32_t)g.stages) { s = 0; ph ^= 1u; }
    }
    if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
}

// ---- backward weight -----------------------------------------------------------------------------------
//   domega'[8g + o][tap][ci] = sum_p dZ[p][8g + o] X[p + tap][8g + ci],   sum_p dZ[p][8g + o]      (Sec. 3.2.1)
// The same patch stream with two boxes per stage: the X patch and the dZ band, the latter on the same
// virtual-pixel grid (row pitch W + kw - 1, its extra columns lie outside the tensor and arrive as zeros,
// so the products of the halo positions vanish).  Per group and 16 virtual pixels: K = the pixels,
// M = (2 taps x 8 input channels), N = 8 output channels; both operands come out of shared memory with
// transposing ldmatrix loads, and a sixth MMA against a matrix of ones gives sum dZ.  A block keeps one
// 64-channel chunk for its whole life, so the sums stay in registers across its bands; at the end every
// warp writes its group's partial block: part[slot][C][taps 8], bsum[slot][C].
template <bool H>
__global__ void __launch_bounds__(kGThreads) grouped8_wgrad_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                                  const __grid_constant__ CUtensorMap tm_dz,
                                                                  const GroupedGeom g, uint32_t dz_off, int slots,
                                                                  float *__restrict__ part, float *__restrict__ bsum,
                                                                  int *err) {
    extern __shared__ uint8_t grouped_smem_raw[];
    uint8_t *ring = (uint8_t *)(((uintptr_t)grouped_smem_raw + 1023) & ~(uintptr_t)1023);
    GroupedCtl *ctl = (GroupedCtl *)(ring + (size_t)g.stages * g.stage_stride);
    volatile int *abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int taps = g.kh * g.kw, ksteps = (taps + 1) / 2, chunks = g.c / 64;
    // the regions TMA never writes (read-ahead tails, the gap between the two boxes) are read as operands:
    // they have to hold zeros, not whatever the last kernel left there
    for (uint32_t i = threadIdx.x; i < (uint32_t)g.stages * g.stage_stride / 16; i += kGThreads)
        reinterpret_cast<uint4 *>(ring)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 8); }
        ctl->abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async_smem();
    __syncthreads();
    const int cc = (int)(blockIdx.x % (uint32_t)chunks), slot = (int)(blockIdx.x / (uint32_t)chunks);
    const uint32_t items = (uint32_t)g.n * g.tiles_h;          // bands of this chunk
    const uint32_t x_bytes = g.patch_bytes, dz_bytes = (uint32_t)g.R * g.Wt * 128u;
    float acc[kGMaxKSteps][4], accs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int ks = 0; ks < kGMaxKSteps; ++ks) acc[ks][0] = acc[ks][1] = acc[ks][2] = acc[ks][3] = 0.f;
    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&tm_x);
            prefetch_tensormap(&tm_dz);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (uint32_t it = (uint32_t)slot; it < items; it += (uint32_t)slots) {
                const int h0 = (int)(it % (uint32_t)g.tiles_h) * g.R, img = (int)(it / (uint32_t)g.tiles_h);
                if (!mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                uint8_t *dst = ring + (size_t)s * g.stage_stride;
                mbar_arrive_expect_tx(&ctl->full[s], x_bytes + dz_bytes);
                tma_load_4d(dst, &tm_x, &ctl->full[s], cc * 64, g.lower_w, h0 + g.lower_h, img);
                tma_load_4d(dst + dz_off, &tm_dz, &ctl->full[s], cc * 64, 0, h0, img);
                if (++s == (uint32_t)g.stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
        }
        return;
    }
    const int gr = lane >> 2, t = lane & 3;
    // A: matrix 0 = pixels 0-7 of the first tap, 1 = pixels 0-7 of the second, 2 / 3 = pixels 8-15
    const int lm_pix = (lane & 7) + (lane >> 4) * 8, lm_tap = (lane >> 3) & 1;
    int vrow[kGMaxKSteps];
    {
        int r = 0, q = 0;
#pragma unroll
        for (int ks = 0; ks < kGMaxKSteps; ++ks) {
            int r1 = r, q1 = q + 1;
            if (q1 == g.kw) { q1 = 0; ++r1; }
            const bool second = lm_tap && 2 * ks + 1 < taps;   // an absent second tap re-reads the first (its rows are dropped)
            vrow[ks] = lm_pix + (second ? r1 * g.Wt + q1 : r * g.Wt + q);
            r = r1; q = q1 + 1;
            if (q >= g.kw) { q -= g.kw; ++r; }
        }
    }
    const int npix = g.R * g.Wt;
    const uint32_t ones = one_h16(H ? 1 : 0) * 0x10001u;       // 1.0 twice
    uint32_t s = 0, ph = 0;
    bool ok = true;
    for (uint32_t it = (uint32_t)slot; it < items && ok; it += (uint32_t)slots) {
        if (!mbar_wait_bounded(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
        const uint32_t xpatch = smem_u32(ring + (size_t)s * g.stage_stride), dzpatch = xpatch + dz_off;
        for (int v0 = 0; v0 < npix; v0 += 16) {
            uint32_t b0, b1;
            {
                const int v = v0 + (lane & 15);
                ldmatrix_x2_trans(b0, b1, dzpatch + (uint32_t)v * 128u + (uint32_t)((warp ^ (v & 7)) << 4));
            }
            mma_16x8x16_t<H>(accs, ones, ones, ones, ones, b0, b1);
#pragma unroll
            for (int ks = 0; ks < kGMaxKSteps; ++ks) {
                if (ks >= ksteps) break;
                const int v = v0 + vrow[ks];
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(a0, a1, a2, a3, xpatch + (uint32_t)v * 128u + (uint32_t)((warp ^ (v & 7)) << 4));
                mma_16x8x16_t<H>(acc[ks], a0, a1, a2, a3, b0, b1);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[s]);
        if (++s == (uint32_t)g.stages) { s = 0; ph ^= 1u; }
    }
    if (!ok && lane == 0) { atomicOr(err, ERRW_TIMEOUT); ctl->abort_flag = 1; }
    // accumulator registers: (row gr = input channel of the first tap, columns 2t, 2t + 1 = output channels),
    // (row gr + 8 = the same input channel of the second tap)
    const int ch0 = cc * 64 + warp * 8, kdim = taps * 8;
    float *prow0 = part + ((size_t)slot * g.c + ch0 + 2 * t) * kdim, *prow1 = prow0 + kdim;
#pragma unroll
    for (int ks = 0; ks < kGMaxKSteps; ++ks) {
        if (2 * ks < taps) {
            prow0[(2 * ks) * 8 + gr] = acc[ks][0];
            prow1[(2 * ks) * 8 + gr] = acc[ks][1];
        }
        if (2 * ks + 1 < taps) {
            prow0[(2 * ks + 1) * 8 + gr] = acc[ks][2];
            prow1[(2 * ks + 1) * 8 + gr] = acc[ks][3];
        }
    }
    if (gr == 0) {
        bsum[(size_t)slot * g.c + ch0 + 2 * t] = accs[0];
        bsum[(size_t)slot * g.c + ch0 + 2 * t + 1] = accs[1];
    }
}

// Adds the block partials and forms the parameter gradients (Table 2, Tune row):
//   domega = s domega', dbeta = sum dZ, db = s dbeta, dgamma = r (sum_k domega' omega + dbeta (b - mu_hat)).
// vec3 == NULL: domega = domega', db = sum dZ.  One block per output channel: thread (k, j) adds slots
// j, j + ng, ... of entry k (a slot's kdim <= 80 entries are contiguous, so the loads coalesce), the ng
// slot groups are then added in order, and the last group column does the same for sum dZ.
__global__ void __launch_bounds__(256) grouped8_wgrad_finish_kernel(int c, int kdim, int slots,
                                                                   const float *__restrict__ part,
                                                                   const float *__restrict__ bsum,
                                                                   const __nv_bfloat16 *__restrict__ w,
                                                                   const float *__restrict__ vec3,
                                                                   const float *__restrict__ b,
                                                                   const float *__restrict__ mean,
                                                                   float *__restrict__ dw, float *__restrict__ db,
                                                                   float *__restrict__ dgamma,
                                                                   float *__restrict__ dbeta, int f16) {
    __shared__ float red[256];
    __shared__ float dots[96];
    const int co = blockIdx.x;
    const int ng = 256 / (kdim + 1);                 // slot groups; column kdim of each group sums dZ
    const int k = threadIdx.x % (kdim + 1), j = threadIdx.x / (kdim + 1);
    float sum = 0.f;
    if (j < ng) {
        if (k < kdim)
            for (int sl = j; sl < slots; sl += ng) sum += part[((size_t)sl * c + co) * kdim + k];
        else
            for (int sl = j; sl < slots; sl += ng) sum += bsum[(size_t)sl * c + co];
    }
    red[threadIdx.x] = sum;
    __syncthreads();
    const float s = vec3 ? vec3[co] : 1.f;
    if (threadIdx.x <= kdim) {
        float tot = 0.f;
        for (int jj = 0; jj < ng; ++jj) tot += red[jj * (kdim + 1) + threadIdx.x];
        if (threadIdx.x < kdim) {
            dw[(size_t)co * kdim + threadIdx.x] = s * tot;
            dots[threadIdx.x] = vec3 ? tot * load_h16(w + (size_t)co * kdim + threadIdx.x, f16) : 0.f;
        } else {
            dots[kdim] = tot;                        // sum dZ
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float d = 0.f;
        for (int i = 0; i < kdim; ++i) d += dots[i];
        const float dsum = dots[kdim];
        if (vec3) {
            dbeta[co] = dsum;
            if (db) db[co] = s * dsum;
            dgamma[co] = vec3[2 * c + co] * (d + dsum * ((b ? b[co] : 0.f) - mean[co]));
        } else if (db) {
            db[co] = dsum;
        }
    }
}

// Backward-data operand: wt[8g + ci][taps - 1 - tap][o] = s[8g + o] w[8g + o][tap][ci]
__global__ void __launch_bounds__(256) grouped8_flip_weights_kernel(int c, int taps, const __nv_bfloat16 *__restrict__ w,
                                                                   const float *__restrict__ s_vec,
                                                                   __nv_bfloat16 *__restrict__ wt, int f16) {
    const int total = c * taps * 8;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int o = i & 7, tap_o = (i >> 3) % taps, row = (i >> 3) / taps;   // row = 8g + ci
        const int co = (row & ~7) + o, ci = row & 7, tap = taps - 1 - tap_o;
        reinterpret_cast<uint16_t *>(wt)[i] =
            pack1_h16((s_vec ? s_vec[co] : 1.f) * load_h16(w + ((size_t)co * taps + tap) * 8 + ci, f16), f16);
    }
}

struct GroupedPlan { bool ok = false; GroupedGeom g; size_t smem = 0; unsigned grid = 0; uint32_t dz_off = 0; int bps = 1; };

GroupedPlan plan_grouped8(int n, int h_in, int w_in, int c, int ho, int wo, int kh, int kw, int lower_h, int lower_w,
                          bool with_dz = false) {
    GroupedPlan pl;
    (void)h_in; (void)w_in;
    const int wt = wo + kw - 1;
    if (wt > 256 || wt < 8 || kh * kw > 2 * kGMaxKSteps || c % 64) return pl;
    const int sms = device_sm_count();
    // The compute warps of one block (8, two per scheduler) cannot hide the ldmatrix -> MMA latency on
    // their own, so the bands are kept small enough for two or three blocks per SM.  Estimated time:
    // rounds over the resident blocks x input pixels of a band, derated for the SM being shared.
    double best = -1.0;
    for (int r = 1; r <= ho && r + kh - 1 <= 256; ++r) {
        const int rows_in = r + kh - 1;
        // stage = the box, plus what the last group of tiles reads past it
        const size_t px = (size_t)((r * wt + 16 * kGTiles - 1) / (16 * kGTiles) * (16 * kGTiles)) + (size_t)(kh - 1) * wt + kw;
        const size_t need = px > (size_t)rows_in * wt ? px : (size_t)rows_in * wt;
        size_t stride = (need * 128 + 1023) / 1024 * 1024;
        const size_t dz_off = stride;                          // the dZ band sits behind the X patch
        if (with_dz) stride += ((size_t)((r * wt + 15) / 16 * 16) * 128 + 1023) / 1024 * 1024;
        const int tiles_h = (ho + r - 1) / r;
        const long long items = (long long)n * tiles_h * (c / 64);
        for (int stages = 2; stages <= 4; ++stages) {
            const size_t smem = 1024 + (size_t)stages * stride + sizeof(GroupedCtl);
            if (smem > 220 * 1024) break;
            int bps = (int)((226 * 1024) / (smem + 1024));
            if (bps > 3) bps = 3;
            if (bps < 1) break;
            const long long slots = (long long)sms * bps;
            const double share = bps == 1 ? 1.9 : (bps == 2 ? 1.25 : 1.0);     // time per item relative to 3 blocks per SM
            const double cost = (double)((items + slots - 1) / slots) * bps * (rows_in * (double)wt + 40.0) * share *
                                (stages == 2 ? 1.1 : 1.0);
            if (best < 0 || cost < best) {
                best = cost;
                pl.ok = true;
                pl.g.R = r; pl.g.Wt = wt; pl.g.rows_in = rows_in; pl.g.tiles_h = tiles_h; pl.g.stages = stages;
                pl.g.patch_bytes = (uint32_t)((size_t)rows_in * wt * 128);
                pl.g.stage_stride = (uint32_t)stride;
                pl.dz_off = (uint32_t)dz_off;
                pl.bps = bps;
                pl.smem = smem;
                pl.grid = (unsigned)(items < slots ? items : slots);
            }
        }
    }
    pl.g.n = n; pl.g.ho = ho; pl.g.wo = wo; pl.g.c = c; pl.g.kh = kh; pl.g.kw = kw;
    pl.g.lower_h = lower_h; pl.g.lower_w = lower_w;
    return pl;
}

}  // namespace

bool grouped8_eligible(const Problem &pb) {
    return pb.groups > 1 && pb.cg == 8 && pb.cog == 8 && pb.c_in % 64 == 0 && pb.stride_h == 1 && pb.stride_w == 1 &&
           pb.dil_h == 1 && pb.dil_w == 1 && pb.kh * pb.kw <= 2 * kGMaxKSteps && pb.w_out + pb.kw - 1 <= 256 &&
           pb.w_in + pb.kw - 1 <= 256 && pb.pad_h <= 128 && pb.pad_w <= 128 && pb.p < (1LL << 30) &&
           pb.pin < (1LL << 30);
}

// act: [n][ha][wa][c]; out: [n][ho][wo][c]; w: [c][kh kw][8] (row = output channel of this pass)
static cudaError_t launch_grouped8(int n, int ha, int wa, int c, int ho, int wo, int kh, int kw, int lower_h,
                                   int lower_w, const void *act, const void *w, const float *bias, void *out,
                                   cudaStream_t st) {
    const GroupedPlan pl = plan_grouped8(n, ha, wa, c, ho, wo, kh, kw, lower_h, lower_w);
    if (!pl.ok) return cudaErrorInvalidValue;
    CUtensorMap ta;
    const unsigned long long dims[4] = {(unsigned long long)c, (unsigned long long)wa, (unsigned long long)ha,
                                        (unsigned long long)n};
    const unsigned long long str[4] = {0, (unsigned long long)c * 2, (unsigned long long)wa * c * 2,
                                       (unsigned long long)ha * wa * c * 2};
    const unsigned int box[4] = {64, (unsigned)pl.g.Wt, (unsigned)pl.g.rows_in, 1};
    if (!make_tmap_tiled_bf16(&ta, act, 4, dims, str, box)) return cudaErrorInvalidValue;
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    static PerDevice attr, attr_h;        // (one flag per instantiation)
    if (call_f16()) {
        if ((e = max_dynamic_smem_once(grouped8_conv_kernel<true>, 220 * 1024, &attr_h)) != cudaSuccess) return e;
        grouped8_conv_kernel<true><<<pl.grid, kGThreads, pl.smem, st>>>(ta, pl.g, (const __nv_bfloat16 *)w, bias,
                                                                       (__nv_bfloat16 *)out, err);
        return cudaGetLastError();
    }
    if ((e = max_dynamic_smem_once(grouped8_conv_kernel<false>, 220 * 1024, &attr)) != cudaSuccess) return e;
    grouped8_conv_kernel<false><<<pl.grid, kGThreads, pl.smem, st>>>(ta, pl.g, (const __nv_bfloat16 *)w, bias,
                                                                    (__nv_bfloat16 *)out, err);
    return cudaGetLastError();
}

cudaError_t launch_grouped8_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                                cudaStream_t st) {
    return launch_grouped8(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.kh, pb.kw, -pb.pad_h, -pb.pad_w, x, w,
                           bias, z, st);
}

cudaError_t launch_grouped8_flip_weights(const Problem &pb, const void *w, const float *s_vec, void *wt,
                                         cudaStream_t st) {
    const int total = pb.c_out * pb.kh * pb.kw * 8;
    grouped8_flip_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(pb.c_out, pb.kh * pb.kw, (const __nv_bfloat16 *)w,
                                                                     s_vec, (__nv_bfloat16 *)wt, call_f16());
    return cudaGetLastError();
}

// dX = omega'_rot (*) dZ: the same kernel on the mirrored problem, weights from launch_grouped8_flip_weights
cudaError_t launch_grouped8_dgrad(const Problem &pb, const void *dz, const void *wt, void *dx, cudaStream_t st) {
    return launch_grouped8(pb.n, pb.h_out, pb.w_out, pb.c_out, pb.h_in, pb.w_in, pb.kh, pb.kw, pb.pad_h - (pb.kh - 1),
                           pb.pad_w - (pb.kw - 1), dz, wt, nullptr, dx, st);
}

// Blocks per 64-channel chunk of the backward-weight kernel = partial rows it writes.
static GroupedPlan plan_grouped8_wgrad(const Problem &pb, int *slots) {
    GroupedPlan pl = plan_grouped8(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.kh, pb.kw, -pb.pad_h, -pb.pad_w,
                                   true);
    if (!pl.ok) return pl;
    const int sms = device_sm_count();
    const int chunks = pb.c_in / 64;
    long long per_chunk = (long long)sms * pl.bps / chunks;
    const long long bands = (long long)pb.n * pl.g.tiles_h;
    if (per_chunk > bands) per_chunk = bands;
    if (per_chunk < 1) per_chunk = 1;
    *slots = (int)per_chunk;
    pl.grid = (unsigned)(per_chunk * chunks);
    return pl;
}

int grouped8_wgrad_slots(const Problem &pb) {
    int slots = 0;
    return plan_grouped8_wgrad(pb, &slots).ok ? slots : 0;
}

// part: [slots][C][taps 8] floats, bsum: [slots][C] floats (slots = grouped8_wgrad_slots)
cudaError_t launch_grouped8_wgrad(const Problem &pb, const void *dz, const void *x, float *part, float *bsum,
                                  cudaStream_t st) {
    int slots = 0;
    const GroupedPlan pl = plan_grouped8_wgrad(pb, &slots);
    if (!pl.ok) return cudaErrorInvalidValue;
    CUtensorMap tx, tdz;
    {
        const unsigned long long dims[4] = {(unsigned long long)pb.c_in, (unsigned long long)pb.w_in,
                                            (unsigned long long)pb.h_in, (unsigned long long)pb.n};
        const unsigned long long str[4] = {0, (unsigned long long)pb.c_in * 2, (unsigned long long)pb.w_in * pb.c_in * 2,
                                           (unsigned long long)pb.h_in * pb.w_in * pb.c_in * 2};
        const unsigned int box[4] = {64, (unsigned)pl.g.Wt, (unsigned)pl.g.rows_in, 1};
        if (!make_tmap_tiled_bf16(&tx, x, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const unsigned long long dims[4] = {(unsigned long long)pb.c_out, (unsigned long long)pb.w_out,
                                            (unsigned long long)pb.h_out, (unsigned long long)pb.n};
        const unsigned long long str[4] = {0, (unsigned long long)pb.c_out * 2, (unsigned long long)pb.w_out * pb.c_out * 2,
                                           (unsigned long long)pb.h_out * pb.w_out * pb.c_out * 2};
        const unsigned int box[4] = {64, (unsigned)pl.g.Wt, (unsigned)pl.g.R, 1};
        if (!make_tmap_tiled_bf16(&tdz, dz, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    int *err = nullptr;
    cudaError_t e = error_word_address(&err);
    if (e != cudaSuccess) return e;
    static PerDevice attr, attr_h;
    if (call_f16()) {
        if ((e = max_dynamic_smem_once(grouped8_wgrad_kernel<true>, 220 * 1024, &attr_h)) != cudaSuccess) return e;
        grouped8_wgrad_kernel<true><<<pl.grid, kGThreads, pl.smem, st>>>(tx, tdz, pl.g, pl.dz_off, slots, part, bsum, err);
        return cudaGetLastError();
    }
    if ((e = max_dynamic_smem_once(grouped8_wgrad_kernel<false>, 220 * 1024, &attr)) != cudaSuccess) return e;
    grouped8_wgrad_kernel<false><<<pl.grid, kGThreads, pl.smem, st>>>(tx, tdz, pl.g, pl.dz_off, slots, part, bsum, err);
    return cudaGetLastError();
}

cudaError_t launch_grouped8_wgrad_finish(const Problem &pb, const float *part, const float *bsum, const void *w,
                                         const float *vec3, const float *b, const float *mean, float *dw, float *db,
                                         float *dgamma, float *dbeta, cudaStream_t st) {
    const int slots = grouped8_wgrad_slots(pb);
    if (slots <= 0) return cudaErrorInvalidValue;
    grouped8_wgrad_finish_kernel<<<pb.c_out, 256, 0, st>>>(pb.c_out, pb.kh * pb.kw * 8, slots, part, bsum,
                                                         (const __nv_bfloat16 *)w, vec3, b, mean, dw, db, dgamma, dbeta,
                                                         call_f16());
    return cudaGetLastError();
}

}  // namespace convbn
