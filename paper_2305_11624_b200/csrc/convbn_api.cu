// C ABI of the ConvBN library: host-side validation, workspace planning, kernel selection.
// Every step of every entry point runs in this library's own kernels; there is no CPU path.
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "kernels.h"

using namespace convbn;

namespace {

thread_local const char *t_last_kernel[CONVBN_PHASE_COUNT] = {"none", "none", "none", "none",
                                                              "none", "none", "none", "none"};

// ---- optional per-kernel timing (CUDA events around every launch this library makes) ----------
struct ProfRec { cudaEvent_t a, b; std::string name; };
thread_local char t_prof_tag[96] = "";   // shape key of the API call in progress
thread_local const char *t_prof_phase = "";   // its phase: fwd, bwd_data, bwd_weight (Eval / Deploy: their own names)
struct Profiler {
    bool on = false;
    std::vector<ProfRec> recs;
};
Profiler g_prof;
std::mutex g_prof_mu;
const size_t kProfCap = 1 << 16;

struct ProfScope {
    cudaStream_t st;
    bool live = false;
    ProfRec rec{};
    ProfScope(const char *name, cudaStream_t s) : st(s) {
        if (!g_prof.on) return;
        std::lock_guard<std::mutex> lk(g_prof_mu);
        if (!g_prof.on || g_prof.recs.size() >= kProfCap) return;
        if (cudaEventCreate(&rec.a) != cudaSuccess) return;
        if (cudaEventCreate(&rec.b) != cudaSuccess) { cudaEventDestroy(rec.a); return; }
        rec.name = std::string(name) + "@" + t_prof_tag + "#" + t_prof_phase;
        cudaEventRecord(rec.a, st);
        live = true;
    }
    ~ProfScope() {
        if (!live) return;
        cudaEventRecord(rec.b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.recs.push_back(rec);
    }
};

inline bool aligned(const void *p, size_t a) { return ((uintptr_t)p % a) == 0; }
inline size_t elem_size(int dtype) { return dtype == CONVBN_F32 ? 4 : 2; }

int make_problem(const convbn_desc *d, Problem *pb) {
    if (!d) return CONVBN_EINVAL;
    if (d->n <= 0 || d->c_in <= 0 || d->h_in <= 0 || d->w_in <= 0 || d->c_out <= 0 || d->kh <= 0 ||
        d->kw <= 0 || d->stride_h <= 0 || d->stride_w <= 0 || d->pad_h < 0 || d->pad_w < 0 ||
        d->dil_h <= 0 || d->dil_w <= 0 || d->groups <= 0)
        return CONVBN_EINVAL;
    if (d->c_in % d->groups || d->c_out % d->groups) return CONVBN_EINVAL;
    if (!(d->eps >= 0.0)) return CONVBN_EINVAL;
    const long long eh = (long long)d->h_in + 2LL * d->pad_h - (long long)d->dil_h * (d->kh - 1) - 1;
    const long long ew = (long long)d->w_in + 2LL * d->pad_w - (long long)d->dil_w * (d->kw - 1) - 1;
    if (eh < 0 || ew < 0) return CONVBN_EINVAL;
    // padded extents and filter spans stay inside 2^30, so that every row and column index fits an int
    if ((long long)d->h_in + 2LL * d->pad_h > (1LL << 30) || (long long)d->w_in + 2LL * d->pad_w > (1LL << 30) ||
        (long long)d->dil_h * (d->kh - 1) > (1LL << 30) || (long long)d->dil_w * (d->kw - 1) > (1LL << 30))
        return CONVBN_EINVAL;
    if (d->dtype != CONVBN_F32 && d->dtype != CONVBN_BF16 && d->dtype != CONVBN_F16) return CONVBN_EINVAL;
    if (d->layout != CONVBN_NCHW && d->layout != CONVBN_NHWC) return CONVBN_EINVAL;
    pb->n = d->n; pb->c_in = d->c_in; pb->h_in = d->h_in; pb->w_in = d->w_in;
    pb->c_out = d->c_out; pb->kh = d->kh; pb->kw = d->kw;
    pb->stride_h = d->stride_h; pb->stride_w = d->stride_w; pb->pad_h = d->pad_h; pb->pad_w = d->pad_w;
    pb->dil_h = d->dil_h; pb->dil_w = d->dil_w; pb->groups = d->groups;
    pb->h_out = (int)(eh / d->stride_h) + 1;
    pb->w_out = (int)(ew / d->stride_w) + 1;
    pb->cg = d->c_in / d->groups;
    pb->cog = d->c_out / d->groups;
    const long long kdim = (long long)pb->cg * d->kh * d->kw;
    pb->p = (long long)d->n * pb->h_out * pb->w_out;
    pb->pin = (long long)d->n * d->h_in * d->w_in;
    // keep every element count inside 2^40 and every row inside int
    if (kdim > (1LL << 30) || pb->p * d->c_out > (1LL << 40) || pb->pin * d->c_in > (1LL << 40))
        return CONVBN_EINVAL;
    pb->kdim = (int)kdim;
    pb->eps = (float)d->eps;
    if (g_prof.on)
        snprintf(t_prof_tag, sizeof(t_prof_tag), "n%d_c%d_%dx%d_o%d_k%dx%d_s%d_g%d", d->n, d->c_in,
                 d->h_in, d->w_in, d->c_out, d->kh, d->kw, d->stride_h, d->groups);
    return CONVBN_OK;
}

int check_pair(const convbn_desc *d) {
    if ((d->dtype == CONVBN_F32 && d->layout == CONVBN_NCHW) ||
        (d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC))
        return CONVBN_OK;
    return CONVBN_EUNSUPPORTED;
}

bool stem_path(const convbn_desc *d, const Problem &pb) {
    return d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && stem_eligible(pb);
}

bool grouped_path(const convbn_desc *d, const Problem &pb) {
    return d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && grouped_bd_eligible(pb);
}

// Workspace carve-up of one phase.  Offsets are multiples of 256 bytes.
struct Plan {
    size_t total = 0;
    size_t w_scaled = 0;   // omega' (storage dtype, weight layout)
    size_t partials = 0;   // [splits][C_out][kdim] fp32
    size_t bsum = 0;       // [bsplits][C_out] fp32
    size_t part_g = 0;     // [bsplits][C_out] fp32 (Eval backward)
    size_t dy = 0;         // Eval backward: s dZ, storage dtype
    size_t vec3 = 0;       // Eval forward: [s | beta - mean s | r]
    size_t dotpart = 0;    // [kt][C_out] fp32 (tensor-core weight-gradient path)
    size_t counters = 0;   // C_out / 32 words (fused epilogue)
    int splits = 1, bsplits = 1, bn_splits = 1;
    size_t xpk = 0, wst = 0;   // small-C_in layers: packed input [n][hp][wp][8], expanded weights [C_out][kh][64]
    bool stem = false;
    bool stem_win_wgrad = false;   // stem weight gradient straight from X (window operand), fused epilogue
    size_t wbd = 0;        // block-diagonal expanded weights [C_out][taps][64], storage dtype
    bool umma_wgrad = false, dw_wgrad = false, dw_tma_wgrad = false, grouped_wgrad = false, grouped8_wgrad = false;
    UmmaWgradPlan uw;
};

bool fused_bwd_path(const convbn_desc *d, const Problem &pb) {
    return d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && fused_bwd1x1_eligible(pb);
}

Plan make_plan(const convbn_desc *d, const Problem &pb, int phase) {
    Plan pl;
    if (phase == CONVBN_PHASE_TUNE_BWD) {
        if (!fused_bwd_path(d, pb)) {       // the two passes run side by side: each has its own region
            const Plan a = make_plan(d, pb, CONVBN_PHASE_TUNE_BWD_DATA), b2 = make_plan(d, pb, CONVBN_PHASE_TUNE_BWD_WEIGHT);
            pl.w_scaled = align_up(a.total, 256);          // here: offset of the backward-weight region
            pl.total = pl.w_scaled + b2.total;
            return pl;
        }
        size_t o = 0;
        auto put = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
        pl.uw.splits = fused_bwd1x1_ctas(pb);
        wgrad_epilogue_shape(pb, &pl.uw);
        pl.bsplits = pl.uw.splits;
        pl.partials = put((size_t)pl.uw.splits * pb.c_out * pb.kdim * sizeof(float));
        pl.bsum = put((size_t)pl.uw.splits * pb.c_out * sizeof(float));
        pl.dotpart = put((size_t)pl.uw.kt * pb.c_out * sizeof(float));
        pl.counters = put((size_t)(pb.c_out / 32 + 1) * sizeof(unsigned int));
        pl.total = o;
        return pl;
    }
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    size_t wbytes = (size_t)pb.c_out * pb.kdim * elem_size(d->dtype);
    // the sub-pixel backward-data path of small-C_in layers keeps its (zero-padded) weight matrix there
    if (d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && subpixel_weight_bytes(pb) > wbytes)
        wbytes = subpixel_weight_bytes(pb);
    const size_t wrows = (size_t)pb.c_out * pb.kdim;
    pl.splits = direct_wgrad_splits(pb);
    pl.bsplits = channel_sum_splits(pb);
    pl.bn_splits = pl.bsplits;                      // pixel slices of the Eval-mode BatchNorm backward
    pl.umma_wgrad = d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC &&
                    umma_wgrad_eligible(pb);
    size_t part_bytes = wrows * pl.splits * sizeof(float), dot_bytes = 0;
    pl.dw_wgrad = d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && dw_eligible(pb) &&
                  dw_wgrad_supported(pb);
    if (pl.dw_wgrad) {
        pl.splits = dw_wgrad_splits(pb);
        part_bytes = wrows * pl.splits * sizeof(float);
        pl.dw_tma_wgrad = dw_tma_eligible(pb);
        if (pl.dw_tma_wgrad && dw_tma_wgrad_partial_bytes(pb) > part_bytes) part_bytes = dw_tma_wgrad_partial_bytes(pb);
    }
    pl.stem = stem_path(d, pb);
    const size_t xpk_bytes = pl.stem ? stem_packed_bytes(pb) : 0, wst_bytes = pl.stem ? stem_weight_bytes(pb) : 0;
    const bool grouped = grouped_path(d, pb);
    const size_t wbd_bytes = grouped ? (size_t)pb.c_out * pb.kh * pb.kw * 64 * elem_size(d->dtype) : 0;
    pl.grouped_wgrad = grouped;
    if (grouped) {
        pl.uw = umma_wgrad_plan(pb);
        pl.bsplits = pl.uw.splits;
        part_bytes = (size_t)pl.uw.splits * (pb.c_out / 64) * pb.kh * pb.kw * 64 * 64 * sizeof(float);
        const int slots = grouped8_eligible(pb) ? grouped8_wgrad_slots(pb) : 0;
        if (slots > 0) {
            pl.grouped8_wgrad = true;
            pl.bsplits = slots;
            part_bytes = (size_t)slots * wrows * sizeof(float);
        }
    }
    if (pl.stem) {
        pl.umma_wgrad = false;
        pl.uw = stem_wgrad_plan(pb);
        pl.bsplits = pl.uw.splits;
        part_bytes = (size_t)pl.uw.splits * stem_krows(pb) * 64 * pb.c_out * sizeof(float);
        if (stem_window_wgrad_eligible(pb)) {
            pl.stem_win_wgrad = true;
            pl.uw = UmmaWgradPlan();
            pl.uw.splits = stem_window_wgrad_ctas(pb);
            wgrad_epilogue_shape(pb, &pl.uw);
            pl.bsplits = pl.uw.splits;
            part_bytes = wrows * pl.uw.splits * sizeof(float);
            dot_bytes = (size_t)pl.uw.kt * pb.c_out * sizeof(float);
        }
    }
    if (pl.umma_wgrad) {
        pl.uw = umma_wgrad_plan(pb);
        pl.bsplits = pl.uw.splits;
        part_bytes = wrows * pl.uw.splits * sizeof(float);
        dot_bytes = (size_t)pl.uw.kt * pb.c_out * sizeof(float);
    }
    switch (phase) {
        case CONVBN_PHASE_TUNE_FWD:
        case CONVBN_PHASE_TUNE_BWD_DATA:
            pl.w_scaled = take(wbytes);
            pl.wbd = take(wbd_bytes);
            if (phase == CONVBN_PHASE_TUNE_FWD) { pl.xpk = take(xpk_bytes); pl.wst = take(wst_bytes); }
            break;
        case CONVBN_PHASE_DEPLOY_FWD:
            pl.wbd = take(wbd_bytes);
            pl.xpk = take(xpk_bytes); pl.wst = take(wst_bytes);
            break;
        case CONVBN_PHASE_DEPLOY_BWD:
            pl.w_scaled = take(wbytes);
            pl.wbd = take(wbd_bytes);
            pl.xpk = take(xpk_bytes);
            pl.partials = take(part_bytes);
            pl.bsum = take((size_t)pl.bsplits * pb.c_out * sizeof(float));
            pl.dotpart = take(dot_bytes);
            pl.counters = take(dot_bytes ? (size_t)(pb.c_out / 32 + 1) * sizeof(unsigned int) : 0);
            break;
        case CONVBN_PHASE_TUNE_BWD_WEIGHT:
            pl.xpk = take(xpk_bytes);
            pl.partials = take(part_bytes);
            pl.bsum = take((size_t)pl.bsplits * pb.c_out * sizeof(float));
            pl.dotpart = take(dot_bytes);
            pl.counters = take(dot_bytes ? (size_t)(pb.c_out / 32 + 1) * sizeof(unsigned int) : 0);
            break;
        case CONVBN_PHASE_EVAL_FWD:
            pl.vec3 = take(3 * (size_t)pb.c_out * sizeof(float));
            pl.wbd = take(wbd_bytes);
            pl.xpk = take(xpk_bytes); pl.wst = take(wst_bytes);
            break;
        case CONVBN_PHASE_EVAL_BWD:
            pl.dy = take((size_t)pb.p * pb.c_out * elem_size(d->dtype));
            pl.w_scaled = take(wbytes);
            pl.wbd = take(wbd_bytes);
            pl.xpk = take(xpk_bytes);
            pl.part_g = take((size_t)pl.bn_splits * pb.c_out * sizeof(float));
            pl.bsum = take((size_t)(pl.bn_splits > pl.bsplits ? pl.bn_splits : pl.bsplits) * pb.c_out * sizeof(float));
            pl.partials = take(part_bytes);
            pl.dotpart = take(dot_bytes);
            pl.counters = take(dot_bytes ? (size_t)(pb.c_out / 32 + 1) * sizeof(unsigned int) : 0);
            break;
        default:
            break;
    }
    pl.total = off;
    return pl;
}

// Device arena of the host-buffer entry point: every tensor of one block plus saved + workspace.
struct HostArena {
    size_t total = 0, x = 0, dz = 0, w = 0, b = 0, gamma = 0, beta = 0, mean = 0, var = 0, z = 0, dx = 0,
           dw = 0, db = 0, dgamma = 0, dbeta = 0, saved = 0, ws = 0;
    size_t x_bytes = 0, z_bytes = 0, w_bytes = 0, dw_bytes = 0, ws_bytes = 0;
};

HostArena make_host_arena(const convbn_desc *d, const Problem &pb) {
    HostArena a;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t es = elem_size(d->dtype), vb = (size_t)pb.c_out * sizeof(float);
    a.x_bytes = (size_t)pb.pin * pb.c_in * es;
    a.z_bytes = (size_t)pb.p * pb.c_out * es;
    a.w_bytes = (size_t)pb.c_out * pb.kdim * es;
    a.dw_bytes = (size_t)pb.c_out * pb.kdim * sizeof(float);
    a.x = take(a.x_bytes); a.dz = take(a.z_bytes); a.w = take(a.w_bytes);
    a.b = take(vb); a.gamma = take(vb); a.beta = take(vb); a.mean = take(vb); a.var = take(vb);
    a.z = take(a.z_bytes); a.dx = take(a.x_bytes); a.dw = take(a.dw_bytes);
    a.db = take(vb); a.dgamma = take(vb); a.dbeta = take(vb);
    a.saved = take(3 * vb);
    for (int ph = CONVBN_PHASE_TUNE_FWD; ph <= CONVBN_PHASE_TUNE_BWD_WEIGHT; ++ph) {
        const size_t t = make_plan(d, pb, ph).total;
        if (t > a.ws_bytes) a.ws_bytes = t;
    }
    a.ws = take(a.ws_bytes);
    a.total = off;
    return a;
}

int check_ws(const Plan &pl, const void *ws, size_t ws_bytes) {
    if (pl.total == 0) return CONVBN_OK;
    if (!ws || ws_bytes < pl.total) return CONVBN_EWORKSPACE;
    if (!aligned(ws, 256)) return CONVBN_EALIGN;
    return CONVBN_OK;
}

#define LAUNCH(name, call) do { ProfScope _ps(name, st); if ((call) != cudaSuccess) return CONVBN_ECUDA; } while (0)
#define CK(expr) do { int _s = (expr); if (_s != CONVBN_OK) return _s; } while (0)
#define CU(expr) do { if ((expr) != cudaSuccess) return CONVBN_ECUDA; } while (0)

inline char *at(void *ws, size_t off) { return (char *)ws + off; }

bool dw_path(const convbn_desc *d, const Problem &pb) {
    return d->dtype == CONVBN_BF16 && d->layout == CONVBN_NHWC && dw_eligible(pb);
}

// Tensor-core eligibility of the forward convolution and its GEMM shape.
bool umma_fwd_shape(const convbn_desc *d, const Problem &pb, UmmaConvShape *s) {
    if (d->dtype != CONVBN_BF16 || d->layout != CONVBN_NHWC || pb.groups != 1) return false;
    *s = UmmaConvShape{pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.c_out, pb.kh, pb.kw,
                       -pb.pad_h, -pb.pad_w, pb.stride_h, pb.stride_w, pb.dil_h, pb.dil_w};
    return umma_conv_eligible(*s);
}

// Backward data as a stride-1 convolution of dZ with the rotated, channel-swapped omega'.
bool umma_dgrad_shape(const convbn_desc *d, const Problem &pb, UmmaConvShape *s) {
    if (d->dtype != CONVBN_BF16 || d->layout != CONVBN_NHWC || pb.groups != 1) return false;
    if (pb.stride_h != 1 || pb.stride_w != 1) return false;
    *s = UmmaConvShape{pb.n, pb.h_out, pb.w_out, pb.c_out, pb.h_in, pb.w_in, pb.c_in, pb.kh, pb.kw,
                       pb.pad_h - (pb.kh - 1) * pb.dil_h, pb.pad_w - (pb.kw - 1) * pb.dil_w, 1, 1, pb.dil_h,
                       pb.dil_w};
    return umma_conv_eligible(*s);
}

// Taps of one residue class of a strided backward-data pass (unit dilation): r = r_max - stride m for
// m = 0 .. count-1, read at output offset off_min + m relative to the class coordinate.
struct ClassTaps { int count, r_max, off_min; };
ClassTaps class_taps(int a, int pad, int k, int stride) {
    ClassTaps c{0, 0, 0};
    const int r0 = (a + pad) % stride;                 // smallest tap with (a + pad - r) divisible by stride
    if (r0 >= k) return c;
    c.count = (k - 1 - r0) / stride + 1;
    c.r_max = r0 + (c.count - 1) * stride;
    c.off_min = (a + pad - c.r_max) / stride;          // exact, may be negative
    return c;
}

bool strided_dgrad_ok(const convbn_desc *d, const Problem &pb) {
    if (d->dtype != CONVBN_BF16 || d->layout != CONVBN_NHWC || pb.groups != 1) return false;
    if (pb.stride_h == 1 && pb.stride_w == 1) return false;
    if (pb.dil_h != 1 || pb.dil_w != 1 || pb.stride_h > 4 || pb.stride_w > 4) return false;
    return pb.c_out % 64 == 0 && pb.c_in % 8 == 0 && pb.c_in >= 64 && pb.c_in <= 4096 &&
           pb.pin < (1LL << 31) - 256;
}

// CONVBN_F16 calls.  IEEE half is an NHWC storage type like bf16 and runs on the same kernels, each of which either
// moves 16-bit elements without looking at them or knows the type (a run-time flag or a second instantiation).
// The descriptor is checked, then the call proceeds as its bf16 twin with the half flag set for the
// launchers (operand format of the MMAs, conversions of results and of rescaled weights, the constant 1, the
// element type of the templated kernels).  The flag is cleared when the call returns.
struct HalfCall {
    convbn_desc d;
    const convbn_desc *use;
    int status = CONVBN_OK;
    bool set_here = false;         // an entry point called from another one must not clear the caller's flag
    explicit HalfCall(const convbn_desc *desc) : use(desc) {
        if (!desc || desc->dtype != CONVBN_F16) return;
        d = *desc;
        d.dtype = CONVBN_BF16;
        use = &d;
        Problem pb;
        status = make_problem(&d, &pb);
        if (status != CONVBN_OK) return;
        if (d.layout != CONVBN_NHWC) { status = CONVBN_EUNSUPPORTED; return; }
        set_call_f16(1);
        set_here = true;
    }
    ~HalfCall() { if (set_here) set_call_f16(0); }
};

// Forward convolution with whatever weights / bias the mode folded: tensor cores when eligible.
int run_conv_fwd(const convbn_desc *d, const Problem &pb, const void *x, const void *w, const float *bias,
                 void *z, const Plan &pl, void *ws, cudaStream_t st, const char **which) {
    UmmaConvShape s;
    void *wbd_scratch = at(ws, pl.wbd);
    if (pl.stem && stem_window_eligible(pb)) {
        // few input channels, stride 2: input rows staged once, windows formed by the operand addressing
        LAUNCH("stem_fwd", launch_stem_window_fwd(pb, x, w, bias, z, st));
        *which = "umma-stem";
    } else if (pl.stem) {
        // few input channels: repack X (8 channels per pixel, zero border) and run the tensor-core GEMM
        // with one 64-wide K row (8 pixels x 8 channels) per filter row
        LAUNCH("stem_pack", launch_stem_pack(pb, x, at(ws, pl.xpk), st));
        LAUNCH("stem_expand", launch_stem_expand_weights(pb, w, nullptr, at(ws, pl.wst), st));
        LAUNCH("stem_fwd", launch_stem_fwd(pb, at(ws, pl.xpk), at(ws, pl.wst), bias, z, st));
        *which = "umma-stem";
    } else if (grouped_path(d, pb) && grouped8_eligible(pb)) {
        // 8 channels per group: warp-level MMAs on the (already folded) weights as they are
        LAUNCH("grouped_fwd", launch_grouped8_fwd(pb, x, w, bias, z, st));
        *which = "grouped-mma";
    } else if (grouped_path(d, pb)) {
        // block-diagonal GEMM: expand the (already folded) weights, then the dense tensor-core kernel
        s = UmmaConvShape{pb.n, pb.h_in, pb.w_in, pb.c_in, pb.h_out, pb.w_out, pb.c_out, pb.kh, pb.kw,
                          -pb.pad_h, -pb.pad_w, pb.stride_h, pb.stride_w, pb.dil_h, pb.dil_w, 1};
        if (!umma_conv_eligible(s)) return CONVBN_EUNSUPPORTED;
        LAUNCH("expand_blockdiag", launch_expand_blockdiag(pb, w, nullptr, wbd_scratch, false, st));
        if (umma_strip_eligible(s))
            LAUNCH("grouped_fwd", launch_umma_strip_conv(s, x, wbd_scratch, bias, z, st));
        else
            LAUNCH("grouped_fwd", launch_umma_conv(s, x, wbd_scratch, bias, z, st));
        *which = "grouped-umma";
    } else if (umma_fwd_shape(d, pb, &s)) {
        if (umma_strip_eligible(s)) {
            LAUNCH("strip_fwd", launch_umma_strip_conv(s, x, w, bias, z, st));
            *which = "umma-strip";
        } else {
            LAUNCH("umma_fwd", launch_umma_conv(s, x, w, bias, z, st));
            *which = "umma";
        }
    } else if (dw_path(d, pb)) {
        LAUNCH("dw_fwd", launch_dw_fwd(pb, x, w, bias, z, st));
        *which = "depthwise";
    } else {
        LAUNCH("direct_fwd", launch_direct_fwd(pb, d->dtype, d->layout, x, w, bias, z, st));
        *which = "direct";
    }
    return CONVBN_OK;
}

// Backward data.  `scale` (C_out floats or NULL) is folded into the weights on the way:
// w_scratch receives omega' in the layout the chosen kernel wants.
int run_conv_dgrad(const convbn_desc *d, const Problem &pb, const void *dz, const void *w, const float *scale,
                   void *w_scratch, void *wbd_scratch, void *dx, cudaStream_t st, const char **which,
                   const float *out_bias = nullptr, bool *bias_done = nullptr) {
    // out_bias (C_in floats, optional): added to dX by the paths whose epilogue can do it; *bias_done says whether it was
    // (the transposed-convolution forward pass is this pass plus a bias)
    if (bias_done) *bias_done = false;
    UmmaConvShape s;
    if (stem_path(d, pb) && stem_window_dgrad_eligible(pb)) {
        // stride 2, C_in <= 4: scatter GEMM over dZ rows, window positions added up on chip
        LAUNCH("stem_dgrad", launch_stem_window_dgrad(pb, dz, w, scale, dx, st));
        *which = "umma-stem";
    } else if (stem_path(d, pb) && subpixel_dgrad_shape(pb, &s) && umma_strip_eligible(s)) {
        // stride 2, C_in <= 4: one stride-1 convolution over dZ whose 16 output columns are the four
        // parity classes of the input position
        LAUNCH("subpixel_weights", launch_subpixel_weights(pb, w, scale, w_scratch, st));
        LAUNCH("stem_dgrad", launch_umma_strip_conv(s, dz, w_scratch, nullptr, dx, st));
        *which = "umma-subpixel";
    } else if (stem_path(d, pb) && stem_dgrad_eligible(pb)) {
        LAUNCH("stem_dgrad", launch_stem_dgrad(pb, dz, w, scale, dx, st));
        *which = "stem-mma";
    } else if (grouped_path(d, pb) && grouped8_eligible(pb)) {
        LAUNCH("grouped_flip", launch_grouped8_flip_weights(pb, w, scale, wbd_scratch, st));
        LAUNCH("grouped_dgrad", launch_grouped8_dgrad(pb, dz, wbd_scratch, dx, st));
        *which = "grouped-mma";
    } else if (grouped_path(d, pb) && pb.stride_h == 1 && pb.stride_w == 1) {
        s = UmmaConvShape{pb.n, pb.h_out, pb.w_out, pb.c_out, pb.h_in, pb.w_in, pb.c_in, pb.kh, pb.kw,
                          pb.pad_h - (pb.kh - 1) * pb.dil_h, pb.pad_w - (pb.kw - 1) * pb.dil_w, 1, 1, pb.dil_h,
                          pb.dil_w, 1};
        if (!umma_conv_eligible(s)) return CONVBN_EUNSUPPORTED;
        LAUNCH("expand_blockdiag", launch_expand_blockdiag(pb, w, scale, wbd_scratch, true, st));
        if (umma_strip_eligible(s))
            LAUNCH("grouped_dgrad", launch_umma_strip_conv(s, dz, wbd_scratch, nullptr, dx, st));
        else
            LAUNCH("grouped_dgrad", launch_umma_conv(s, dz, wbd_scratch, nullptr, dx, st));
        *which = "grouped-umma";
    } else if (strided_dgrad_ok(d, pb) && subpixel_wide_shape(pb, &s) && umma_strip_eligible(s)) {
        // stride 2: the four parity classes of the input position as column blocks of ONE stride-1
        // convolution over dZ (one launch, the dZ patch staged once, absent taps skipped)
        LAUNCH("subpixel_weights", launch_subpixel_weights(pb, w, scale, w_scratch, st));
        LAUNCH("strip_dgrad", launch_umma_strip_conv(s, dz, w_scratch, nullptr, dx, st));
        *which = "umma-subpixel";
    } else if (strided_dgrad_ok(d, pb)) {
        // Strided backward data, one stride-1 GEMM per residue class (a, b) of the input position:
        // rows h = stride_h i + a only meet taps r with (a + pad_h - r) divisible by stride_h, at output
        // row i + (a + pad_h - r) / stride_h; no multiplication by inserted zeros.
        bool any_empty = false;
        for (int a = 0; a < pb.stride_h && !any_empty; ++a) any_empty = class_taps(a, pb.pad_h, pb.kh, pb.stride_h).count == 0;
        for (int b2 = 0; b2 < pb.stride_w && !any_empty; ++b2) any_empty = class_taps(b2, pb.pad_w, pb.kw, pb.stride_w).count == 0;
        if (any_empty &&
            cudaMemsetAsync(dx, 0, (size_t)pb.pin * pb.c_in * elem_size(d->dtype), st) != cudaSuccess)
            return CONVBN_ECUDA;
        // one launch writes every class's weight matrix (when the kernel has at most 64 taps)
        const bool merged = pb.kh * pb.kw <= 64;
        if (merged) {
            ClassTapTable where;
            memset(&where, 0, sizeof(where));
            size_t eoff = 0;
            for (int a = 0; a < pb.stride_h && a < pb.h_in; ++a)
                for (int b2 = 0; b2 < pb.stride_w && b2 < pb.w_in; ++b2) {
                    const ClassTaps ch = class_taps(a, pb.pad_h, pb.kh, pb.stride_h);
                    const ClassTaps cw = class_taps(b2, pb.pad_w, pb.kw, pb.stride_w);
                    if (ch.count == 0 || cw.count == 0) continue;
                    for (int mh = 0; mh < ch.count; ++mh)
                        for (int mw = 0; mw < cw.count; ++mw) {
                            const int tap = (ch.r_max - pb.stride_h * mh) * pb.kw + (cw.r_max - pb.stride_w * mw);
                            where.offset[tap] = (long long)eoff;
                            where.count[tap] = ch.count * cw.count;
                            where.pos[tap] = mh * cw.count + mw;
                        }
                    eoff += (size_t)ch.count * cw.count * pb.c_in * pb.c_out;
                }
            LAUNCH("reparam_dgrad", launch_reparam_dgrad_classes(pb, w, scale, w_scratch, where, st));
        }
        size_t woff = 0;
        for (int a = 0; a < pb.stride_h && a < pb.h_in; ++a)
            for (int b2 = 0; b2 < pb.stride_w && b2 < pb.w_in; ++b2) {
                const ClassTaps ch = class_taps(a, pb.pad_h, pb.kh, pb.stride_h);
                const ClassTaps cw = class_taps(b2, pb.pad_w, pb.kw, pb.stride_w);
                if (ch.count == 0 || cw.count == 0) continue;
                char *wc = (char *)w_scratch + woff;
                woff += (size_t)ch.count * cw.count * pb.c_in * pb.c_out * elem_size(d->dtype);
                UmmaConvShape cs{pb.n, pb.h_out, pb.w_out, pb.c_out,
                                 (pb.h_in - a + pb.stride_h - 1) / pb.stride_h,
                                 (pb.w_in - b2 + pb.stride_w - 1) / pb.stride_w, pb.c_in, ch.count, cw.count,
                                 ch.off_min, cw.off_min, 1, 1, 1, 1, 0};
                cs.out_sn = (long long)pb.h_in * pb.w_in * pb.c_in;
                cs.out_sh = pb.stride_h * pb.w_in * pb.c_in;
                cs.out_sw = pb.stride_w * pb.c_in;
                if (!umma_conv_eligible(cs)) return CONVBN_EUNSUPPORTED;
                if (!merged)
                    LAUNCH("reparam_dgrad", launch_reparam_dgrad_class(pb, w, scale, wc, ch.count, cw.count, ch.r_max,
                                                                       cw.r_max, pb.stride_h, pb.stride_w, st));
                LAUNCH("umma_dgrad", launch_umma_conv(cs, dz, wc, nullptr,
                                                      (char *)dx + ((size_t)a * pb.w_in + b2) * pb.c_in *
                                                                       elem_size(d->dtype), st));
            }
        *which = "umma-strided";
    } else if (umma_dgrad_shape(d, pb, &s)) {
        LAUNCH("reparam_dgrad", launch_reparam_dgrad(pb, w, scale, w_scratch, st));
        if (umma_strip_eligible(s)) {
            LAUNCH("strip_dgrad", launch_umma_strip_conv(s, dz, w_scratch, out_bias, dx, st));
            *which = "umma-strip";
        } else {
            LAUNCH("umma_dgrad", launch_umma_conv(s, dz, w_scratch, out_bias, dx, st));
            *which = "umma";
        }
        if (bias_done && out_bias) *bias_done = true;
    } else if (dw_path(d, pb)) {
        if (pb.stride_h == 1 && pb.stride_w == 1) {
            // dX = omega'_rot (*) dZ is itself a stride-1 depthwise convolution of dZ with the rotated
            // taps and padding (k-1) d - p: run the forward kernel on the mirrored problem.
            Problem mp = pb;
            mp.h_in = pb.h_out; mp.w_in = pb.w_out; mp.h_out = pb.h_in; mp.w_out = pb.w_in;
            mp.pad_h = (pb.kh - 1) * pb.dil_h - pb.pad_h; mp.pad_w = (pb.kw - 1) * pb.dil_w - pb.pad_w;
            mp.p = pb.pin; mp.pin = pb.p;
            if (dw_tma_eligible(mp)) {
                // the streaming kernel scales and reverses the taps itself
                LAUNCH("dw_dgrad", launch_dw_tma(mp, dz, w, nullptr, dx, st, nullptr, scale, true));
            } else {
                LAUNCH("rescale_weight", launch_rescale_weight(pb, d->dtype, w, scale, w_scratch, st, true));
                LAUNCH("dw_dgrad", launch_dw_fwd(mp, dz, w_scratch, nullptr, dx, st));
            }
        } else {
            const void *wd = w;
            if (scale) {
                LAUNCH("rescale_weight", launch_rescale_weight(pb, d->dtype, w, scale, w_scratch, st));
                wd = w_scratch;
            }
            LAUNCH("dw_dgrad", launch_dw_dgrad(pb, dz, wd, dx, st));
        }
        *which = "depthwise";
    } else {
        const void *wd = w;
        if (scale) {
            LAUNCH("rescale_weight", launch_rescale_weight(pb, d->dtype, w, scale, w_scratch, st));
            wd = w_scratch;
        }
        LAUNCH("direct_dgrad", launch_direct_dgrad(pb, d->dtype, d->layout, dz, wd, dx, st));
        *which = "direct";
    }
    return CONVBN_OK;
}

// Parameter gradients from dZ and X, shared by all modes.
//   vec3 != NULL (Tune): dw = s domega', dbeta, db = s dbeta, dgamma          (Table 2, Tune row)
//   vec3 == NULL        : dw = domega', db = sum dZ if db != NULL               (Deploy / Eval rows)
int run_param_grads(const convbn_desc *d, const Problem &pb, const Plan &pl, const void *dz, const void *x,
                    const void *w, const float *vec3, const float *b, const float *mean, float *dw, float *db,
                    float *dgamma, float *dbeta, void *ws, cudaStream_t st, const char **which) {
    float *partials = (float *)at(ws, pl.partials), *bsum = (float *)at(ws, pl.bsum);
    const bool need_bsum = vec3 || db;
    const bool tc = pl.grouped_wgrad || pl.umma_wgrad || pl.stem;   // tensor-core paths sum dZ inside the GEMM
    if (need_bsum && !tc && !pl.dw_tma_wgrad)
        LAUNCH("channel_sum", launch_channel_sum_partial(pb, d->dtype, d->layout, dz, bsum, pl.bsplits, st));
    if (pl.stem_win_wgrad) {
        float *dotpart = (float *)at(ws, pl.dotpart);
        unsigned int *counters = (unsigned int *)at(ws, pl.counters);
        LAUNCH("stem_wgrad", launch_stem_window_wgrad(pb, dz, x, partials, bsum, counters, st));
        LAUNCH("wgrad_epilogue_fused", launch_wgrad_epilogue_fused(pb, pl.uw, partials, bsum, w, vec3, b, mean, dw,
                                                                   dotpart, counters, db, dgamma, dbeta, need_bsum,
                                                                   st));
        *which = "umma-stem";
    } else if (pl.stem) {
        LAUNCH("stem_pack", launch_stem_pack(pb, x, at(ws, pl.xpk), st));
        LAUNCH("stem_wgrad", launch_stem_wgrad(pb, pl.uw, dz, at(ws, pl.xpk), partials, bsum, st));
        LAUNCH("wgrad_epilogue_stem", launch_wgrad_epilogue_stem(pb, pl.uw, partials, bsum, w, vec3, b, mean, dw, db,
                                                                 dgamma, dbeta, need_bsum, st));
        *which = "umma-stem";
    } else if (pl.grouped8_wgrad) {
        LAUNCH("grouped_wgrad", launch_grouped8_wgrad(pb, dz, x, partials, bsum, st));
        LAUNCH("grouped_wgrad_finish", launch_grouped8_wgrad_finish(pb, partials, bsum, w, vec3, b, mean, dw, db,
                                                                    dgamma, dbeta, st));
        *which = "grouped-mma";
    } else if (pl.grouped_wgrad) {
        LAUNCH("grouped_wgrad", launch_umma_wgrad(pb, pl.uw, dz, x, partials, bsum, nullptr, st));
        LAUNCH("wgrad_epilogue_bd", launch_wgrad_epilogue_bd(pb, partials, pl.uw.splits, need_bsum ? bsum : nullptr,
                                                             need_bsum ? pl.bsplits : 0, w, vec3, b, mean, dw, db,
                                                             dgamma, dbeta, st));
        *which = "grouped-umma";
    } else if (pl.umma_wgrad) {
        float *dotpart = (float *)at(ws, pl.dotpart);
        unsigned int *counters = (unsigned int *)at(ws, pl.counters);
        LAUNCH("umma_wgrad", launch_umma_wgrad(pb, pl.uw, dz, x, partials, bsum, counters, st));
        LAUNCH("wgrad_epilogue_fused", launch_wgrad_epilogue_fused(pb, pl.uw, partials, bsum, w, vec3, b, mean, dw,
                                                                   dotpart, counters, db, dgamma, dbeta, need_bsum,
                                                                   st));
        *which = "umma";
    } else if (pl.dw_tma_wgrad) {
        int nparts = 0;
        LAUNCH("dw_wgrad", launch_dw_tma_wgrad(pb, dz, x, partials, &nparts, st));
        LAUNCH("dw_wgrad_finish", launch_dw_wgrad_finish(pb, partials, nparts, w, vec3, b, mean, dw, db, dgamma, dbeta, st));
        *which = "depthwise";
    } else {
        if (pl.dw_wgrad)
            LAUNCH("dw_wgrad", launch_dw_wgrad(pb, dz, x, partials, pl.splits, st));
        else
            LAUNCH("direct_wgrad", launch_direct_wgrad(pb, d->dtype, d->layout, dz, x, partials, pl.splits, st));
        LAUNCH("wgrad_epilogue", launch_wgrad_epilogue(pb, d->dtype, partials, pl.splits, need_bsum ? bsum : nullptr,
                                                       need_bsum ? pl.bsplits : 0, w, vec3, b, mean, dw, db, dgamma,
                                                       dbeta, st));
        *which = pl.dw_wgrad ? "depthwise" : "direct";
    }
    return CONVBN_OK;
}

}  // namespace

extern "C" {

int convbn_out_shape(const convbn_desc *desc, int *h_out, int *w_out) {
    Problem pb;
    if (!h_out || !w_out) return CONVBN_EINVAL;
    CK(make_problem(desc, &pb));
    *h_out = pb.h_out;
    *w_out = pb.w_out;
    return CONVBN_OK;
}

int convbn_linear_desc(int rows, int in_features, int out_features, int dtype, double eps, convbn_desc *desc) {
    if (!desc || rows <= 0 || in_features <= 0 || out_features <= 0 || !(eps >= 0.0)) return CONVBN_EINVAL;
    if (dtype != CONVBN_F32 && dtype != CONVBN_BF16 && dtype != CONVBN_F16) return CONVBN_EINVAL;
    memset(desc, 0, sizeof(*desc));
    desc->n = rows; desc->c_in = in_features; desc->h_in = 1; desc->w_in = 1;
    desc->c_out = out_features; desc->kh = 1; desc->kw = 1;
    desc->stride_h = desc->stride_w = desc->dil_h = desc->dil_w = desc->groups = 1;
    desc->dtype = dtype;
    desc->layout = dtype == CONVBN_F32 ? CONVBN_NCHW : CONVBN_NHWC;
    desc->eps = eps;
    return CONVBN_OK;
}

size_t convbn_saved_bytes(const convbn_desc *desc, int mode) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return 0;
    desc = half.use;
    Problem pb;
    if (make_problem(desc, &pb) != CONVBN_OK) return 0;
    switch (mode) {
        case CONVBN_MODE_TUNE: return 3 * (size_t)pb.c_out * sizeof(float);
        case CONVBN_MODE_EVAL: return (size_t)pb.p * pb.c_out * elem_size(desc->dtype);
        default: return 0;
    }
}

size_t convbn_workspace_bytes(const convbn_desc *desc, int phase) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return 0;
    desc = half.use;
    Problem pb;
    if (phase < 0 || phase >= CONVBN_PHASE_COUNT) return 0;
    if (make_problem(desc, &pb) != CONVBN_OK) return 0;
    return make_plan(desc, pb, phase).total;
}

int convbn_tune_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b,
                    const float *gamma, const float *beta, const float *run_mean,
                    const float *run_var, void *z, void *saved, void *workspace,
                    size_t workspace_bytes, void *stream) {
    HalfCall half(desc);              // CONVBN_F16: checked here, then run as the 16-bit path with the half flag set
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "fwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!x || !w || !gamma || !beta || !run_mean || !run_var || !z || !saved) return CONVBN_EINVAL;
    if (!aligned(x, 16) || !aligned(w, 16) || !aligned(z, 16) || !aligned(saved, 16) ||
        !aligned(b, 4) || !aligned(gamma, 4) || !aligned(beta, 4) || !aligned(run_mean, 4) ||
        !aligned(run_var, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_TUNE_FWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    float *vec3 = (float *)saved;
    void *wf = at(workspace, pl.w_scaled);
    UmmaConvShape us;
    if (pl.stem && stem_window_eligible(pb)) {
        const BnFold fold{gamma, beta, run_mean, run_var, b, pb.eps, vec3};
        LAUNCH("stem_fwd", launch_stem_window_fwd(pb, x, w, nullptr, z, st, &fold));
        t_last_kernel[CONVBN_PHASE_TUNE_FWD] = "umma-stem";
        return CONVBN_OK;
    }
    if (pl.stem) {
        const BnFold fold{gamma, beta, run_mean, run_var, b, pb.eps, vec3};
        LAUNCH("stem_pack", launch_stem_pack(pb, x, at(workspace, pl.xpk), st));
        LAUNCH("stem_expand", launch_stem_expand_weights(pb, w, nullptr, at(workspace, pl.wst), st));
        LAUNCH("stem_fwd", launch_stem_fwd(pb, at(workspace, pl.xpk), at(workspace, pl.wst), nullptr, z, st, &fold));
        t_last_kernel[CONVBN_PHASE_TUNE_FWD] = "umma-stem";
        return CONVBN_OK;
    }
    if (!grouped_path(desc, pb) && umma_fwd_shape(desc, pb, &us)) {
        // dense tensor-core path: s, b' and the saved vectors are formed inside the GEMM kernel and s is
        // applied to the fp32 accumulator, so one launch does the whole forward pass
        const BnFold fold{gamma, beta, run_mean, run_var, b, pb.eps, vec3};
        if (umma_strip_eligible(us)) {
            LAUNCH("strip_fwd", launch_umma_strip_conv(us, x, w, nullptr, z, st, &fold));
            t_last_kernel[CONVBN_PHASE_TUNE_FWD] = "umma-strip";
        } else {
            LAUNCH("umma_fwd", launch_umma_conv(us, x, w, nullptr, z, st, &fold));
            t_last_kernel[CONVBN_PHASE_TUNE_FWD] = "umma";
        }
        return CONVBN_OK;
    }
    if (dw_path(desc, pb) && dw_tma_eligible(pb)) {
        // depthwise 3x3: the fold is formed inside the streaming kernel from the raw weights
        const BnFold fold{gamma, beta, run_mean, run_var, b, pb.eps, vec3};
        LAUNCH("dw_fwd", launch_dw_tma(pb, x, w, nullptr, z, st, &fold));
        t_last_kernel[CONVBN_PHASE_TUNE_FWD] = "depthwise";
        return CONVBN_OK;
    }
    LAUNCH("reparam", launch_reparam(pb, desc->dtype, desc->layout, w, b, gamma, beta, run_mean, run_var, vec3, wf,
                      nullptr, st));
    CK(run_conv_fwd(desc, pb, x, wf, vec3 + pb.c_out, z, pl, workspace, st, &t_last_kernel[CONVBN_PHASE_TUNE_FWD]));
    return CONVBN_OK;
}

int convbn_tune_bwd_data(const convbn_desc *desc, const void *dz, const void *w, const void *saved,
                         void *dx, void *workspace, size_t workspace_bytes, void *stream) {
    HalfCall half(desc);              // CONVBN_F16: checked here, then run as the 16-bit path with the half flag set
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "bwd_data";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!dz || !w || !saved || !dx) return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(w, 16) || !aligned(saved, 16) || !aligned(dx, 16))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_TUNE_BWD_DATA);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    void *wf = at(workspace, pl.w_scaled);
    CK(run_conv_dgrad(desc, pb, dz, w, (const float *)saved, wf, at(workspace, pl.wbd), dx, st,
                      &t_last_kernel[CONVBN_PHASE_TUNE_BWD_DATA]));
    return CONVBN_OK;
}

int convbn_tune_bwd_weight(const convbn_desc *desc, const void *dz, const void *x, const void *w,
                           const float *b, const float *run_mean, const void *saved, float *dw,
                           float *db, float *dgamma, float *dbeta, void *workspace,
                           size_t workspace_bytes, void *stream) {
    HalfCall half(desc);              // CONVBN_F16: checked here, then run as the 16-bit path with the half flag set
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "bwd_weight";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!dz || !x || !w || !run_mean || !saved || !dw || !dgamma || !dbeta) return CONVBN_EINVAL;
    if ((b == nullptr) != (db == nullptr)) return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(x, 16) || !aligned(w, 16) || !aligned(saved, 16) ||
        !aligned(dw, 16) || !aligned(b, 4) || !aligned(run_mean, 4) || !aligned(db, 4) ||
        !aligned(dgamma, 4) || !aligned(dbeta, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_TUNE_BWD_WEIGHT);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    CK(run_param_grads(desc, pb, pl, dz, x, w, (const float *)saved, b, run_mean, dw, db, dgamma, dbeta,
                       workspace, st, &t_last_kernel[CONVBN_PHASE_TUNE_BWD_WEIGHT]));
    return CONVBN_OK;
}

}  // extern "C"

namespace {
// Side lane of convbn_tune_bwd: one stream and two events per device and host thread, made on first use.  The
// parameter-gradient pass (GEMM + epilogue) runs there while the input-gradient pass (weight re-layout + GEMM) runs
// on the caller's stream; the caller's stream waits for the lane before the call returns, so stream order is what
// the caller sees.  (Per thread: two threads sharing the events could wait on each other's fork points.)
struct SideLane {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool pending = false;          // passes begun there that no stream has joined yet
};
thread_local SideLane t_side_lane[kMaxDevices];

int side_lane(SideLane **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CONVBN_ECUDA;
    SideLane &l = t_side_lane[dev];
    if (!l.stream) {
        if (cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) != cudaSuccess) { l.stream = nullptr; return CONVBN_ECUDA; }
        if (cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming) != cudaSuccess)
            return CONVBN_ECUDA;
    }
    *out = &l;
    return CONVBN_OK;
}

// `side(lane stream)` and `main_pass()` side by side, the caller's stream joined to the lane before return.
// Under the profiler (per-kernel event pairs on one stream) they run one after the other.
template <class Side, class Main>
int side_by_side(cudaStream_t st, Side &&side, Main &&main_pass) {
    if (g_prof.on) {
        CK(main_pass());
        return side(st);
    }
    SideLane *lane = nullptr;
    CK(side_lane(&lane));
    CU(cudaEventRecord(lane->fork, st));
    CU(cudaStreamWaitEvent(lane->stream, lane->fork, 0));
    const int ss = side(lane->stream);
    // whatever happened on the lane, the caller's stream joins it again (a capture must not be left forked)
    const bool joined = cudaEventRecord(lane->join, lane->stream) == cudaSuccess;
    const int sm = main_pass();
    if (!joined || cudaStreamWaitEvent(st, lane->join, 0) != cudaSuccess) return CONVBN_ECUDA;
    return ss != CONVBN_OK ? ss : sm;
}
}  // namespace

extern "C" {
static int tune_bwd_impl(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                         const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                         float *dbeta, void *workspace, size_t workspace_bytes, void *stream, bool defer_join) {
    HalfCall half(desc);              // CONVBN_F16: checked here, then run as the 16-bit path with the half flag set
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "bwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!dz || !x || !w || !run_mean || !saved || !dx || !dw || !dgamma || !dbeta) return CONVBN_EINVAL;
    if ((b == nullptr) != (db == nullptr)) return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(x, 16) || !aligned(w, 16) || !aligned(saved, 16) || !aligned(dx, 16) ||
        !aligned(dw, 16) || !aligned(b, 4) || !aligned(run_mean, 4) || !aligned(db, 4) || !aligned(dgamma, 4) ||
        !aligned(dbeta, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_TUNE_BWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    if (!fused_bwd_path(desc, pb)) {
        void *ws_w = workspace ? at(workspace, pl.w_scaled) : nullptr;
        const size_t bytes_d = pl.w_scaled, bytes_w = pl.total - pl.w_scaled;
        t_last_kernel[CONVBN_PHASE_TUNE_BWD] = "two-calls";
        if (g_prof.on) {                 // per-kernel timing wants one stream, deferred or not
            CK(convbn_tune_bwd_data(desc, dz, w, saved, dx, workspace, bytes_d, stream));
            return convbn_tune_bwd_weight(desc, dz, x, w, b, run_mean, saved, dw, db, dgamma, dbeta, ws_w, bytes_w, stream);
        }
        SideLane *lane = nullptr;
        CK(side_lane(&lane));
        cudaStream_t st = (cudaStream_t)stream;
        CU(cudaEventRecord(lane->fork, st));
        CU(cudaStreamWaitEvent(lane->stream, lane->fork, 0));
        const int sw = convbn_tune_bwd_weight(desc, dz, x, w, b, run_mean, saved, dw, db, dgamma, dbeta, ws_w, bytes_w,
                                              lane->stream);
        // whatever happened on the lane, the caller's stream joins it again (a capture must not be left forked)
        const bool joined = cudaEventRecord(lane->join, lane->stream) == cudaSuccess;
        const int sd = convbn_tune_bwd_data(desc, dz, w, saved, dx, workspace, bytes_d, stream);
        if (!joined) return CONVBN_ECUDA;
        if (defer_join) lane->pending = true;
        else if (cudaStreamWaitEvent(st, lane->join, 0) != cudaSuccess) return CONVBN_ECUDA;
        return sw != CONVBN_OK ? sw : sd;
    }
    cudaStream_t st = (cudaStream_t)stream;
    float *partials = (float *)at(workspace, pl.partials), *bsum = (float *)at(workspace, pl.bsum);
    float *dotpart = (float *)at(workspace, pl.dotpart);
    unsigned int *counters = (unsigned int *)at(workspace, pl.counters);
    const float *vec3 = (const float *)saved;
    LAUNCH("umma_bwd", launch_fused_bwd1x1(pb, dz, x, w, vec3, dx, partials, bsum, counters, st));
    t_last_kernel[CONVBN_PHASE_TUNE_BWD] = "umma-fused-bwd";
    if (defer_join && !g_prof.on) {
        // dX is complete on the caller's stream; the parameter gradients are finished on the side lane
        SideLane *lane = nullptr;
        CK(side_lane(&lane));
        CU(cudaEventRecord(lane->fork, st));
        CU(cudaStreamWaitEvent(lane->stream, lane->fork, 0));
        cudaStream_t st = lane->stream;
        LAUNCH("wgrad_epilogue_fused", launch_wgrad_epilogue_fused(pb, pl.uw, partials, bsum, w, vec3, b, run_mean, dw,
                                                                   dotpart, counters, db, dgamma, dbeta, true, st));
        CU(cudaEventRecord(lane->join, lane->stream));
        lane->pending = true;
        return CONVBN_OK;
    }
    LAUNCH("wgrad_epilogue_fused", launch_wgrad_epilogue_fused(pb, pl.uw, partials, bsum, w, vec3, b, run_mean, dw, dotpart,
                                                               counters, db, dgamma, dbeta, true, st));
    return CONVBN_OK;
}

int convbn_tune_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                    const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                    float *dbeta, void *workspace, size_t workspace_bytes, void *stream) {
    return tune_bwd_impl(desc, dz, x, w, b, run_mean, saved, dx, dw, db, dgamma, dbeta, workspace, workspace_bytes, stream,
                         false);
}

int convbn_tune_bwd_begin(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                          const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                          float *dbeta, void *workspace, size_t workspace_bytes, void *stream) {
    return tune_bwd_impl(desc, dz, x, w, b, run_mean, saved, dx, dw, db, dgamma, dbeta, workspace, workspace_bytes, stream,
                         true);
}

int convbn_tune_bwd_join(void *stream) {
    SideLane *lane = nullptr;
    CK(side_lane(&lane));
    // the lane is one stream: its last join point covers every pass begun before it.  With nothing pending the
    // lane is left alone (inside a stream capture it may not be part of the capture at all).
    if (lane->pending) {
        CU(cudaEventRecord(lane->join, lane->stream));
        CU(cudaStreamWaitEvent((cudaStream_t)stream, lane->join, 0));
        lane->pending = false;
    }
    return CONVBN_OK;
}

int convbn_eval_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b,
                    const float *gamma, const float *beta, const float *run_mean,
                    const float *run_var, void *z, void *y_saved, void *workspace,
                    size_t workspace_bytes, void *stream) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "eval_fwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!x || !w || !gamma || !beta || !run_mean || !run_var || !z || !y_saved) return CONVBN_EINVAL;
    if (!aligned(x, 16) || !aligned(w, 16) || !aligned(z, 16) || !aligned(y_saved, 16) ||
        !aligned(b, 4) || !aligned(gamma, 4) || !aligned(beta, 4) || !aligned(run_mean, 4) ||
        !aligned(run_var, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_EVAL_FWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    float *vec3 = (float *)at(workspace, pl.vec3);
    // BN acts on Y, which already holds the conv bias: shift = beta - mean s
    LAUNCH("reparam", launch_reparam(pb, desc->dtype, desc->layout, w, nullptr, gamma, beta, run_mean, run_var, vec3,
                      nullptr, nullptr, st));
    CK(run_conv_fwd(desc, pb, x, w, b, y_saved, pl, workspace, st, &t_last_kernel[CONVBN_PHASE_EVAL_FWD]));
    LAUNCH("bn_eval_fwd", launch_bn_eval_fwd(pb, desc->dtype, desc->layout, y_saved, vec3, z, st));
    return CONVBN_OK;
}

int convbn_eval_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *y_saved,
                    const void *w, const float *gamma, const float *run_mean, const float *run_var,
                    void *dx, float *dw, float *db, float *dgamma, float *dbeta, void *workspace,
                    size_t workspace_bytes, void *stream) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "eval_bwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!dz || !x || !y_saved || !w || !gamma || !run_mean || !run_var || !dx || !dw || !dgamma || !dbeta)
        return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(x, 16) || !aligned(y_saved, 16) || !aligned(w, 16) ||
        !aligned(dx, 16) || !aligned(dw, 16) || !aligned(gamma, 4) || !aligned(run_mean, 4) ||
        !aligned(run_var, 4) || !aligned(db, 4) || !aligned(dgamma, 4) || !aligned(dbeta, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_EVAL_BWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    void *dy = at(workspace, pl.dy);
    float *pg = (float *)at(workspace, pl.part_g), *pbm = (float *)at(workspace, pl.bsum);
    LAUNCH("bn_eval_bwd", launch_bn_eval_bwd(pb, desc->dtype, desc->layout, dz, y_saved, gamma, run_mean, run_var, dy, pg,
                          pbm, pl.bn_splits, st));
    LAUNCH("bn_eval_finish", launch_bn_eval_finish(pb, pg, pbm, pl.bn_splits, gamma, run_var, db, dgamma, dbeta, st));
    // dX and domega both start from dY and use separate regions of the workspace: side by side, as in Tune mode
    return side_by_side(
        st,
        [&](cudaStream_t lane) {
            const char *unused = nullptr;
            return run_param_grads(desc, pb, pl, dy, x, w, nullptr, nullptr, nullptr, dw, nullptr, nullptr, nullptr, workspace,
                                   lane, &unused);
        },
        [&]() {
            return run_conv_dgrad(desc, pb, dy, w, nullptr, at(workspace, pl.w_scaled), at(workspace, pl.wbd), dx, st,
                                  &t_last_kernel[CONVBN_PHASE_EVAL_BWD]);
        });
}

int convbn_deploy_prepare(const convbn_desc *desc, const void *w, const float *b, const float *gamma,
                          const float *beta, const float *run_mean, const float *run_var,
                          void *w_fused, float *b_fused, void *stream) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "deploy_prepare";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!w || !gamma || !beta || !run_mean || !run_var || !w_fused || !b_fused) return CONVBN_EINVAL;
    if (!aligned(w, 16) || !aligned(w_fused, 16) || !aligned(b, 4) || !aligned(gamma, 4) ||
        !aligned(beta, 4) || !aligned(run_mean, 4) || !aligned(run_var, 4) || !aligned(b_fused, 4))
        return CONVBN_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    LAUNCH("reparam", launch_reparam(pb, desc->dtype, desc->layout, w, b, gamma, beta, run_mean, run_var, nullptr,
                      w_fused, b_fused, st));
    return CONVBN_OK;
}

int convbn_deploy_fwd(const convbn_desc *desc, const void *x, const void *w_fused,
                      const float *b_fused, void *z, void *workspace, size_t workspace_bytes,
                      void *stream) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "deploy_fwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!x || !w_fused || !b_fused || !z) return CONVBN_EINVAL;
    if (!aligned(x, 16) || !aligned(w_fused, 16) || !aligned(z, 16) || !aligned(b_fused, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_DEPLOY_FWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    CK(run_conv_fwd(desc, pb, x, w_fused, b_fused, z, pl, workspace, st, &t_last_kernel[CONVBN_PHASE_DEPLOY_FWD]));
    return CONVBN_OK;
}

int convbn_deploy_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *w_fused,
                      void *dx, float *dw_fused, float *db_fused, void *workspace,
                      size_t workspace_bytes, void *stream) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    t_prof_phase = "deploy_bwd";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!dz || !x || !w_fused || !dx || !dw_fused || !db_fused) return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(x, 16) || !aligned(w_fused, 16) || !aligned(dx, 16) ||
        !aligned(dw_fused, 16) || !aligned(db_fused, 4))
        return CONVBN_EALIGN;
    const Plan pl = make_plan(desc, pb, CONVBN_PHASE_DEPLOY_BWD);
    CK(check_ws(pl, workspace, workspace_bytes));
    cudaStream_t st = (cudaStream_t)stream;
    return side_by_side(
        st,
        [&](cudaStream_t lane) {
            const char *unused = nullptr;
            return run_param_grads(desc, pb, pl, dz, x, w_fused, nullptr, nullptr, nullptr, dw_fused, db_fused, nullptr, nullptr,
                                   workspace, lane, &unused);
        },
        [&]() {
            return run_conv_dgrad(desc, pb, dz, w_fused, nullptr, at(workspace, pl.w_scaled), at(workspace, pl.wbd), dx, st,
                                  &t_last_kernel[CONVBN_PHASE_DEPLOY_BWD]);
        });
}

// ---- TransposedConv-BN -----------------------------------------------------------------------------
namespace {

// The convolution a transposed convolution transposes: its input is the transposed layer's OUTPUT.
struct TconvView {
    convbn_desc conv;          // descriptor of that convolution
    Problem pb;                // and its problem
    int h_out, w_out;          // output extent of the transposed layer
    size_t wcount;             // weight elements
    size_t off_w, off_zero, off_dwp, off_bsum, off_inner, total;
    int bsplits;
    Problem sum_pb;            // a 1x1 problem whose output is the transposed layer's output (for the channel sums)
    Plan fwd, bwd;             // plans of the inner convolution: plain forward, plain backward
};

int tconv_view(const convbn_desc *d, TconvView *v) {
    if (!d) return CONVBN_EINVAL;
    if (d->n <= 0 || d->c_in <= 0 || d->h_in <= 0 || d->w_in <= 0 || d->c_out <= 0 || d->kh <= 0 || d->kw <= 0 ||
        d->stride_h <= 0 || d->stride_w <= 0 || d->pad_h < 0 || d->pad_w < 0 || d->dil_h <= 0 || d->dil_w <= 0 ||
        d->groups <= 0)
        return CONVBN_EINVAL;
    const long long ho = (long long)(d->h_in - 1) * d->stride_h - 2LL * d->pad_h + (long long)d->dil_h * (d->kh - 1) + 1;
    const long long wo = (long long)(d->w_in - 1) * d->stride_w - 2LL * d->pad_w + (long long)d->dil_w * (d->kw - 1) + 1;
    if (ho <= 0 || wo <= 0 || ho > (1 << 24) || wo > (1 << 24)) return CONVBN_EINVAL;
    v->h_out = (int)ho; v->w_out = (int)wo;
    v->conv = *d;
    v->conv.c_in = d->c_out; v->conv.c_out = d->c_in; v->conv.h_in = (int)ho; v->conv.w_in = (int)wo;
    CK(make_problem(&v->conv, &v->pb));
    CK(check_pair(&v->conv));
    if (v->pb.h_out != d->h_in || v->pb.w_out != d->w_in) return CONVBN_EINVAL;
    convbn_desc one = *d;
    one.c_in = d->c_out; one.h_in = (int)ho; one.w_in = (int)wo; one.kh = one.kw = 1;
    one.stride_h = one.stride_w = one.dil_h = one.dil_w = 1; one.pad_h = one.pad_w = 0; one.groups = 1;
    CK(make_problem(&one, &v->sum_pb));
    v->bsplits = channel_sum_splits(v->sum_pb);
    v->fwd = make_plan(&v->conv, v->pb, CONVBN_PHASE_DEPLOY_FWD);
    v->bwd = make_plan(&v->conv, v->pb, CONVBN_PHASE_DEPLOY_BWD);
    v->wcount = (size_t)d->c_in * (d->c_out / d->groups) * d->kh * d->kw;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at0 = off; off += (bytes + 255) / 256 * 256; return at0; };
    v->off_w = take(v->wcount * elem_size(d->dtype));
    v->off_zero = take((size_t)d->c_in * sizeof(float));
    v->off_dwp = take(v->wcount * sizeof(float));
    v->off_bsum = take((size_t)v->bsplits * d->c_out * sizeof(float));
    v->off_inner = off;
    v->total = off + (v->fwd.total > v->bwd.total ? v->fwd.total : v->bwd.total);
    return CONVBN_OK;
}

// An IEEE-half transposed layer runs as its bf16 twin: `twin` receives the descriptor to use from here on and
// `inner` the convolution it transposes, typed half again, for HalfCall to check and to set the call's flag.
int tconv_open(const convbn_desc *&desc, convbn_desc *twin, convbn_desc *inner, TconvView *v) {
    if (!desc) return CONVBN_EINVAL;
    const bool is_half = desc->dtype == CONVBN_F16;
    if (is_half) { *twin = *desc; twin->dtype = CONVBN_BF16; desc = twin; }
    CK(tconv_view(desc, v));
    *inner = v->conv;
    if (is_half) inner->dtype = CONVBN_F16;
    return CONVBN_OK;
}

}  // namespace

int convbn_tconv_out_shape(const convbn_desc *desc, int *h_out, int *w_out) {
    TconvView v;
    convbn_desc twin, inner_desc;
    CK(tconv_open(desc, &twin, &inner_desc, &v));
    if (!h_out || !w_out) return CONVBN_EINVAL;
    *h_out = v.h_out; *w_out = v.w_out;
    return CONVBN_OK;
}

size_t convbn_tconv_workspace_bytes(const convbn_desc *desc) {
    TconvView v;
    convbn_desc twin, inner_desc;
    if (tconv_open(desc, &twin, &inner_desc, &v) != CONVBN_OK) return 0;
    HalfCall half(&inner_desc);
    return half.status == CONVBN_OK ? v.total : 0;
}

int convbn_tconv_tune_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b, const float *gamma,
                          const float *beta, const float *run_mean, const float *run_var, void *z, void *saved,
                          void *workspace, size_t workspace_bytes, void *stream) {
    TconvView v;
    convbn_desc twin, inner_desc;
    t_prof_phase = "tconv_fwd";
    CK(tconv_open(desc, &twin, &inner_desc, &v));
    HalfCall half(&inner_desc);            // CONVBN_F16: the inner convolution's paths are checked, the half flag is set
    if (half.status != CONVBN_OK) return half.status;
    if (!x || !w || !gamma || !beta || !run_mean || !run_var || !z || !saved) return CONVBN_EINVAL;
    if (!aligned(x, 16) || !aligned(w, 16) || !aligned(z, 16) || !aligned(saved, 16) || !aligned(b, 4) ||
        !aligned(gamma, 4) || !aligned(beta, 4) || !aligned(run_mean, 4) || !aligned(run_var, 4))
        return CONVBN_EALIGN;
    if (!workspace || workspace_bytes < v.total) return CONVBN_EWORKSPACE;
    if (!aligned(workspace, 256)) return CONVBN_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const bool nhwc = desc->layout == CONVBN_NHWC;
    const int taps = desc->kh * desc->kw, cig = desc->c_in / desc->groups, cog = desc->c_out / desc->groups;
    float *vec3 = (float *)saved;
    void *wf = at(workspace, v.off_w), *inner = at(workspace, v.off_inner);
    LAUNCH("tconv_vec3", launch_tconv_vec3(desc->c_out, (float)desc->eps, b, gamma, beta, run_mean, run_var, vec3, st));
    LAUNCH("tconv_rescale", launch_tconv_rescale(desc->dtype, nhwc, (long long)v.wcount, taps, cig, cog, w, vec3, wf, st));
    // Z = omega' scattered over X: the backward-data pass of the convolution with the same weights
    const char *which = nullptr;
    bool bias_done = false;          // unit-stride tensor-core layers add b' in the GEMM's own epilogue (one rounding)
    CK(run_conv_dgrad(&v.conv, v.pb, x, wf, nullptr, at(inner, v.bwd.w_scaled), at(inner, v.bwd.wbd), z, st, &which,
                      vec3 + desc->c_out, &bias_done));
    if (!bias_done) {
        const long long count = (long long)desc->n * desc->c_out * v.h_out * v.w_out;
        LAUNCH("tconv_bias", launch_tconv_bias(desc->dtype, nhwc, count, desc->c_out, (long long)v.h_out * v.w_out,
                                               vec3 + desc->c_out, z, st));
    }
    return CONVBN_OK;
}

int convbn_tconv_tune_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                          const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                          float *dbeta, void *workspace, size_t workspace_bytes, void *stream) {
    TconvView v;
    convbn_desc twin, inner_desc;
    t_prof_phase = "tconv_bwd";
    CK(tconv_open(desc, &twin, &inner_desc, &v));
    HalfCall half(&inner_desc);
    if (half.status != CONVBN_OK) return half.status;
    if (!dz || !x || !w || !run_mean || !saved || !dx || !dw || !dgamma || !dbeta) return CONVBN_EINVAL;
    if ((b == nullptr) != (db == nullptr)) return CONVBN_EINVAL;
    if (!aligned(dz, 16) || !aligned(x, 16) || !aligned(w, 16) || !aligned(saved, 16) || !aligned(dx, 16) ||
        !aligned(dw, 16) || !aligned(b, 4) || !aligned(run_mean, 4) || !aligned(db, 4) || !aligned(dgamma, 4) ||
        !aligned(dbeta, 4))
        return CONVBN_EALIGN;
    if (!workspace || workspace_bytes < v.total) return CONVBN_EWORKSPACE;
    if (!aligned(workspace, 256)) return CONVBN_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const bool nhwc = desc->layout == CONVBN_NHWC;
    const int taps = desc->kh * desc->kw, cig = desc->c_in / desc->groups, cog = desc->c_out / desc->groups;
    const float *vec3 = (const float *)saved;
    void *wf = at(workspace, v.off_w), *inner = at(workspace, v.off_inner);
    float *zero = (float *)at(workspace, v.off_zero), *dwp = (float *)at(workspace, v.off_dwp);
    float *bsum = (float *)at(workspace, v.off_bsum);
    // omega' is re-formed from omega and the saved scale (Sec. 3.4: Tune mode keeps X and a few vectors)
    LAUNCH("tconv_rescale", launch_tconv_rescale(desc->dtype, nhwc, (long long)v.wcount, taps, cig, cog, w, vec3, wf, st));
    CU(cudaMemsetAsync(zero, 0, (size_t)desc->c_in * sizeof(float), st));
    // dX gathers dZ through omega': the forward pass of that convolution, without a bias
    const char *which = nullptr;
    CK(run_conv_fwd(&v.conv, v.pb, dz, wf, zero, dx, v.fwd, inner, st, &which));
    // domega' contracts X with windows of dZ: that convolution's weight gradient with the two tensors exchanged
    CK(run_param_grads(&v.conv, v.pb, v.bwd, x, dz, wf, nullptr, nullptr, nullptr, dwp, nullptr, nullptr, nullptr, inner,
                       st, &which));
    LAUNCH("channel_sum", launch_channel_sum_partial(v.sum_pb, desc->dtype, desc->layout, dz, bsum, v.bsplits, st));
    LAUNCH("tconv_epilogue", launch_tconv_param_epilogue(desc->dtype, nhwc, desc->c_out, taps, cig, cog, dwp, w, vec3, b,
                                                         run_mean, bsum, v.bsplits, dw, db, dgamma, dbeta, st));
    return CONVBN_OK;
}

int convbn_check(void *stream) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return CONVBN_ECUDA;
    int word = 0;
    if (read_and_clear_error_word(&word) != cudaSuccess) return CONVBN_ECUDA;
    return (word & ERRW_TIMEOUT) ? CONVBN_ETIMEOUT : CONVBN_OK;
}

static int glue_call(int mode, int dtype, const void *a, const void *b, void *out, long long count, void *stream) {
    if (count < 0 || (dtype != CONVBN_F32 && dtype != CONVBN_BF16 && dtype != CONVBN_F16)) return CONVBN_EINVAL;
    if (count == 0) return CONVBN_OK;
    if (!a || !out || (mode != 0 && !b)) return CONVBN_EINVAL;
    if (!aligned(a, 16) || !aligned(out, 16) || !aligned(b, 16)) return CONVBN_EALIGN;
    return launch_glue(mode, dtype, a, b, out, count, (cudaStream_t)stream) == cudaSuccess ? CONVBN_OK : CONVBN_ECUDA;
}
int convbn_relu(int dtype, const void *a, void *out, long long count, void *stream) {
    return glue_call(0, dtype, a, nullptr, out, count, stream);
}
int convbn_add_relu(int dtype, const void *a, const void *b, void *out, long long count, void *stream) {
    return glue_call(1, dtype, a, b, out, count, stream);
}
int convbn_relu_bwd(int dtype, const void *a, const void *y, void *out, long long count, void *stream) {
    return glue_call(2, dtype, a, y, out, count, stream);
}
int convbn_add(int dtype, const void *a, const void *b, void *out, long long count, void *stream) {
    return glue_call(3, dtype, a, b, out, count, stream);
}

int convbn_selftest_wait_timeout(void *stream) {
    if (launch_selftest_wait_timeout(100000ull, (cudaStream_t)stream) != cudaSuccess) return CONVBN_ECUDA;
    return CONVBN_OK;
}

int convbn_profile_begin(void) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    for (auto &r : g_prof.recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    g_prof.recs.clear();
    g_prof.on = true;
    return CONVBN_OK;
}

int convbn_profile_end(char *report, size_t report_bytes) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof.on = false;
    int status = CONVBN_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) status = CONVBN_ECUDA;
    std::map<std::string, std::pair<long long, double>> agg;
    for (auto &r : g_prof.recs) {
        float ms = 0.f;
        if (status == CONVBN_OK && cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) {
            auto &e = agg[r.name];
            e.first += 1;
            e.second += ms;
        }
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    g_prof.recs.clear();
    if (report && report_bytes) {
        size_t off = 0;
        report[0] = 0;
        for (auto &kv : agg) {
            int n = snprintf(report + off, report_bytes - off, "%s %lld %.6f\n", kv.first.c_str(),
                             kv.second.first, kv.second.second);
            if (n < 0 || (size_t)n >= report_bytes - off) { report[off] = 0; break; }
            off += (size_t)n;
        }
    }
    return status;
}

size_t convbn_host_step_arena_bytes(const convbn_desc *desc) {
    HalfCall half(desc);
    if (half.status != CONVBN_OK) return 0;
    desc = half.use;
    Problem pb;
    if (make_problem(desc, &pb) != CONVBN_OK) return 0;
    return make_host_arena(desc, pb).total;
}

namespace {
// Copy lanes of convbn_tune_step_host: an upload stream, a download stream and their events, per device and host
// thread, made on first use.  Inputs go up on one lane, results come down on the other, the kernels run on the
// caller's stream in between; both directions of the bus are then busy at once, within a call (dZ goes up while Z
// comes down) and, when the caller defers the join, across calls (the next layer's X goes up while this layer's dX
// comes down).
struct CopyLanes {
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t start = nullptr, in = nullptr, dz = nullptr, fwd = nullptr, bwd = nullptr, done = nullptr;
    const void *last_arena = nullptr;     // the previous call's arena: a call that reuses it waits for its downloads
    bool pending = false;                 // downloads no stream has joined yet
};
thread_local CopyLanes t_copy_lanes[kMaxDevices];

int copy_lanes(CopyLanes **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CONVBN_ECUDA;
    CopyLanes &l = t_copy_lanes[dev];
    if (!l.up) {
        if (cudaStreamCreateWithFlags(&l.up, cudaStreamNonBlocking) != cudaSuccess) { l.up = nullptr; return CONVBN_ECUDA; }
        if (cudaStreamCreateWithFlags(&l.down, cudaStreamNonBlocking) != cudaSuccess) return CONVBN_ECUDA;
        cudaEvent_t *ev[6] = {&l.start, &l.in, &l.dz, &l.fwd, &l.bwd, &l.done};
        for (cudaEvent_t *e : ev)
            if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return CONVBN_ECUDA;
    }
    *out = &l;
    return CONVBN_OK;
}

int host_step_impl(const convbn_desc *desc, const void *x, const void *dz, const void *w, const float *b,
                   const float *gamma, const float *beta, const float *run_mean, const float *run_var, void *z, void *dx,
                   float *dw, float *db, float *dgamma, float *dbeta, void *device_arena, size_t arena_bytes, void *stream,
                   bool defer_join) {
    HalfCall half(desc);              // CONVBN_F16: the step runs as its bf16 twin with the half flag set
    if (half.status != CONVBN_OK) return half.status;
    desc = half.use;
    Problem pb;
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    if (!x || !dz || !w || !gamma || !beta || !run_mean || !run_var || !z || !dx || !dw || !dgamma || !dbeta)
        return CONVBN_EINVAL;
    if ((b == nullptr) != (db == nullptr)) return CONVBN_EINVAL;
    const HostArena ar = make_host_arena(desc, pb);
    if (!device_arena || arena_bytes < ar.total) return CONVBN_EWORKSPACE;
    if (!aligned(device_arena, 256)) return CONVBN_EALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    CopyLanes *ln = nullptr;
    CK(copy_lanes(&ln));
    char *d = (char *)device_arena;
    const size_t vb = (size_t)pb.c_out * sizeof(float);
    auto h2d = [&](size_t off, const void *src, size_t bytes) {
        return cudaMemcpyAsync(d + off, src, bytes, cudaMemcpyHostToDevice, ln->up);
    };
    auto d2h = [&](void *dst, size_t off, size_t bytes) {
        return cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, ln->down);
    };
    // uploads start after everything queued earlier on `stream` (which may still read the arena); an arena that
    // the previous call used is also still being downloaded from
    CU(cudaEventRecord(ln->start, st));
    CU(cudaStreamWaitEvent(ln->up, ln->start, 0));
    if (ln->pending && ln->last_arena == device_arena) CU(cudaStreamWaitEvent(ln->up, ln->done, 0));
    CU(h2d(ar.x, x, ar.x_bytes));
    CU(h2d(ar.w, w, ar.w_bytes));
    CU(h2d(ar.gamma, gamma, vb));
    CU(h2d(ar.beta, beta, vb));
    CU(h2d(ar.mean, run_mean, vb));
    CU(h2d(ar.var, run_var, vb));
    if (b) CU(h2d(ar.b, b, vb));
    CU(cudaEventRecord(ln->in, ln->up));
    CU(h2d(ar.dz, dz, ar.z_bytes));
    CU(cudaEventRecord(ln->dz, ln->up));
    const float *db_dev = b ? (const float *)(d + ar.b) : nullptr;
    CU(cudaStreamWaitEvent(st, ln->in, 0));
    CK(convbn_tune_fwd(desc, d + ar.x, d + ar.w, db_dev, (const float *)(d + ar.gamma), (const float *)(d + ar.beta),
                       (const float *)(d + ar.mean), (const float *)(d + ar.var), d + ar.z, d + ar.saved, d + ar.ws,
                       ar.ws_bytes, stream));
    CU(cudaEventRecord(ln->fwd, st));
    CU(cudaStreamWaitEvent(ln->down, ln->fwd, 0));
    CU(d2h(z, ar.z, ar.z_bytes));
    CU(cudaStreamWaitEvent(st, ln->dz, 0));
    CK(convbn_tune_bwd_data(desc, d + ar.dz, d + ar.w, d + ar.saved, d + ar.dx, d + ar.ws, ar.ws_bytes, stream));
    CK(convbn_tune_bwd_weight(desc, d + ar.dz, d + ar.x, d + ar.w, db_dev, (const float *)(d + ar.mean), d + ar.saved,
                              (float *)(d + ar.dw), b ? (float *)(d + ar.db) : nullptr, (float *)(d + ar.dgamma),
                              (float *)(d + ar.dbeta), d + ar.ws, ar.ws_bytes, stream));
    CU(cudaEventRecord(ln->bwd, st));
    CU(cudaStreamWaitEvent(ln->down, ln->bwd, 0));
    CU(d2h(dx, ar.dx, ar.x_bytes));
    CU(d2h(dw, ar.dw, ar.dw_bytes));
    CU(d2h(dgamma, ar.dgamma, vb));
    CU(d2h(dbeta, ar.dbeta, vb));
    if (db) CU(d2h(db, ar.db, vb));
    CU(cudaEventRecord(ln->done, ln->down));
    ln->last_arena = device_arena;
    ln->pending = true;
    if (!defer_join) {
        CU(cudaStreamWaitEvent(st, ln->done, 0));
        ln->pending = false;
    }
    return CONVBN_OK;
}
}  // namespace

int convbn_tune_step_host(const convbn_desc *desc, const void *x, const void *dz, const void *w,
                          const float *b, const float *gamma, const float *beta,
                          const float *run_mean, const float *run_var, void *z, void *dx, float *dw,
                          float *db, float *dgamma, float *dbeta, void *device_arena,
                          size_t arena_bytes, void *stream) {
    return host_step_impl(desc, x, dz, w, b, gamma, beta, run_mean, run_var, z, dx, dw, db, dgamma, dbeta, device_arena,
                          arena_bytes, stream, false);
}

int convbn_tune_step_host_begin(const convbn_desc *desc, const void *x, const void *dz, const void *w,
                                const float *b, const float *gamma, const float *beta,
                                const float *run_mean, const float *run_var, void *z, void *dx, float *dw,
                                float *db, float *dgamma, float *dbeta, void *device_arena,
                                size_t arena_bytes, void *stream) {
    return host_step_impl(desc, x, dz, w, b, gamma, beta, run_mean, run_var, z, dx, dw, db, dgamma, dbeta, device_arena,
                          arena_bytes, stream, true);
}

int convbn_tune_step_host_join(void *stream) {
    CopyLanes *ln = nullptr;
    CK(copy_lanes(&ln));
    if (ln->pending) {
        CU(cudaStreamWaitEvent((cudaStream_t)stream, ln->done, 0));
        ln->pending = false;
    }
    return CONVBN_OK;
}

// ---- parameter gradients without any caller-provided scratch -------------------------------------
// Built-in scratch of convbn_tune_bwd_weight_noalloc.  It is part of the library image: every GPU
// that loads the library carries these bytes until the process exits.  In host code the name below
// is only a host-side handle of the symbol, never a device address, so the host asks the runtime for
// the real address once per device and hands that to the kernels.
#define CONVBN_NOALLOC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[CONVBN_NOALLOC_SCRATCH_BYTES];

namespace {
const int kMaxDevices = 64;
void *g_noalloc_ptr[kMaxDevices] = {nullptr};
std::mutex g_noalloc_mu;

// Device address of the built-in scratch on the CURRENT device (looked up on first use there).
int noalloc_scratch_address(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CONVBN_ECUDA;
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr)
            return CONVBN_ECUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return CONVBN_OK;
}
}  // namespace

int convbn_tune_bwd_weight_noalloc(const convbn_desc *desc, const void *dz, const void *x,
                                   const void *w, const float *b, const float *run_mean,
                                   const void *saved, float *dw, float *db, float *dgamma,
                                   float *dbeta, void *stream) {
    Problem pb;
    t_prof_phase = "bwd_weight";
    CK(make_problem(desc, &pb));
    CK(check_pair(desc));
    const size_t need = make_plan(desc, pb, CONVBN_PHASE_TUNE_BWD_WEIGHT).total;
    if (need > (size_t)CONVBN_NOALLOC_SCRATCH_BYTES) return CONVBN_ECAPACITY;
    void *scratch = nullptr;
    CK(noalloc_scratch_address(&scratch));
    // Same kernels as convbn_tune_bwd_weight, with the built-in array standing in for the caller's
    // workspace.  Every scratch word those kernels read is written earlier in the same call, so
    // nothing left over from a previous call has to be cleared.
    return convbn_tune_bwd_weight(desc, dz, x, w, b, run_mean, saved, dw, db, dgamma, dbeta, scratch,
                                  (size_t)CONVBN_NOALLOC_SCRATCH_BYTES, stream);
}

const char *convbn_status_string(int status) {
    switch (status) {
        case CONVBN_OK: return "ok";
        case CONVBN_EINVAL: return "invalid descriptor or NULL pointer";
        case CONVBN_EUNSUPPORTED: return "dtype/layout pair not supported";
        case CONVBN_EWORKSPACE: return "workspace missing or too small";
        case CONVBN_EALIGN: return "pointer not aligned as required";
        case CONVBN_ECUDA: return "CUDA call failed";
        case CONVBN_ETIMEOUT: return "a bounded device-side wait expired";
        case CONVBN_ECAPACITY: return "problem needs more scratch than the built-in 16 MiB array holds";
        default: return "unknown status";
    }
}

const char *convbn_last_kernel(int phase) {
    if (phase < 0 || phase >= CONVBN_PHASE_COUNT) return "none";
    return t_last_kernel[phase];
}

}  // extern "C"
