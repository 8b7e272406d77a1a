// Host-side launchers of every kernel family.  Each returns the cudaError_t of its launch.
#pragma once

#include "common.cuh"

namespace convbn {

// ---- per-output-channel reparameterisation (Sec. 3.3 definitions of omega', b') -------------
// Writes, each if its pointer is non-NULL:
//   vec3      : [s | b' | r]  (3 * C_out floats)
//   w_scaled  : omega' in the layout of w, storage dtype
//   b_fused   : b' alone (C_out floats)
// scale_weights = false copies omega unscaled (s = 1 for the weight only; used by Eval mode).
cudaError_t launch_reparam(const Problem &pb, int dtype, int layout, const void *w, const float *b,
                           const float *gamma, const float *beta, const float *mean,
                           const float *var, float *vec3, void *w_scaled, float *b_fused,
                           cudaStream_t st);

// omega' = s omega re-formed from the saved scale vector (first C_out floats of vec3; NULL = 1).
// reverse_row writes each weight row back to front (the 180-degree tap rotation when C_in/G = 1).
cudaError_t launch_rescale_weight(const Problem &pb, int dtype, const void *w, const float *vec3,
                                  void *w_scaled, cudaStream_t st, bool reverse_row = false);

// ---- direct (one thread per output element) convolution kernels, any shape -----------------
cudaError_t launch_direct_fwd(const Problem &pb, int dtype, int layout, const void *x,
                              const void *w, const float *bias, void *z, cudaStream_t st);
cudaError_t launch_direct_dgrad(const Problem &pb, int dtype, int layout, const void *dz,
                                const void *w, void *dx, cudaStream_t st);
int direct_wgrad_splits(const Problem &pb);
// partials: [splits][C_out][kdim] fp32, row order of the weight layout
cudaError_t launch_direct_wgrad(const Problem &pb, int dtype, int layout, const void *dz,
                                const void *x, float *partials, int splits, cudaStream_t st);

// ---- tensor-core implicit-GEMM convolution (bf16 NHWC, groups = 1) -----------------------------
// out[n,ho,wo,:cn] = bias + sum over taps (r,q) and channels c of
//     act[n, lower_h + ho stride_h + r dil_h, lower_w + wo stride_w + q dil_w, c] * wmat[:, (r taps_w + q) ca + c]
// with zeros outside the activation tensor.  wmat is a row-major [cn][taps_h taps_w ca] bf16 matrix.
struct UmmaConvShape {
    int n, ha, wa, ca;       // activation tensor [n][ha][wa][ca]
    int ho, wo, cn;          // output tensor [n][ho][wo][cn]
    int taps_h, taps_w, lower_h, lower_w, stride_h, stride_w, dil_h, dil_w;
    // 1: grouped convolution run as a block-diagonal GEMM: output channels [64 b, 64 b + 64) read only
    // activation channels [64 b, 64 b + 64) and wmat is [cn][taps * 64] (zeros outside a channel's group).
    int blockdiag = 0;
    // Strided output, used when out_sw != 0 (no bias in this mode): output pixel (n, i, j) is written at
    // out + n out_sn + i out_sh + j out_sw (elements) instead of densely.
    long long out_sn = 0;
    int out_sh = 0, out_sw = 0;
    // Sub-pixel output (stride-2 backward data of a layer with at most 4 input channels, strip kernel only,
    // cn = 16): output "pixel" (n, i, j) holds the 2 x 2 input positions (2 i + a, 2 j + b); GEMM column
    // 8 a + b sub_cin + ci is written to out[n][2 i + a][2 j + b][ci] of a [n][sub_hin][sub_win][sub_cin]
    // tensor (positions outside it are dropped).  0: off.
    int sub_cin = 0, sub_hin = 0, sub_win = 0;
    // The same regrouping for wide layers (sub_cin a multiple of 64, cn = 4 sub_cin): GEMM columns
    // [cls sub_cin, (cls + 1) sub_cin), cls = 2 a + b, are the channels of input position (2 i + a, 2 j + b);
    // bit t of sub_mask[cls] says that tap t = tr taps_w + tq has weights for that class (other taps are
    // skipped, not multiplied by zeros).
    unsigned sub_mask[4] = {0, 0, 0, 0};
};
bool umma_conv_eligible(const UmmaConvShape &s);
// BatchNorm parameters for in-kernel reparameterisation: the kernel forms s and b' per output channel,
// computes out = s * (wmat (*) act) + b' and (CTA 0) writes [s | b' | r] to vec3 (3 cn floats, may be NULL).
struct BnFold {
    const float *gamma, *beta, *mean, *var, *b;   // b may be NULL
    float eps;
    float *vec3;
};
// fold != NULL replaces `bias` (dense output mode only).
cudaError_t launch_umma_conv(const UmmaConvShape &s, const void *act, const void *wmat, const float *bias,
                             void *out, cudaStream_t st, const BnFold *fold = nullptr);
// Stride-1 multi-tap convolutions with the input patch staged once per tile (see umma_strip.cu): same
// contract as launch_umma_conv (dense output mode, groups = 1).  Eligibility depends on the image size.
bool umma_strip_eligible(const UmmaConvShape &s);
cudaError_t launch_umma_strip_conv(const UmmaConvShape &s, const void *act, const void *wmat, const float *bias,
                                   void *out, cudaStream_t st, const BnFold *fold = nullptr);
// Backward data of a stride-2 layer with C_in <= 4 as ONE stride-1 convolution over dZ (Sec. 3.2.1: the
// transposed convolution, regrouped by the parity of the input position): the four parity classes of an
// input position become 4 C_in output columns of a GEMM whose taps are the dZ offsets any class needs;
// taps a class does not meet have zero weights.  subpixel_dgrad_shape fills the strip-kernel shape and
// returns false when the layer does not qualify; the weight matrix is [16][taps_h taps_w C_out] bf16,
// row 8 a + b C_in + ci, entry s[co] w[co][r][q][ci] with r = a + pad_h - 2 d (d = the tap's dZ row offset).
bool subpixel_dgrad_shape(const Problem &pb, UmmaConvShape *s);
// Wide variant (C_in, C_out multiples of 64, stride 2): weight matrix [4 C_in][taps_h taps_w C_out], row
// (2 a + b) C_in + ci.  Replaces one GEMM launch per parity class by one launch.
bool subpixel_wide_shape(const Problem &pb, UmmaConvShape *s);
size_t subpixel_weight_bytes(const Problem &pb);
cudaError_t launch_subpixel_weights(const Problem &pb, const void *w, const float *s_vec, void *wsub,
                                    cudaStream_t st);
// Weight operand of the backward-data GEMM: w_t[ci][taps-1-tap][co] = s[co] w[co][tap][ci]
// (s_vec == NULL: unscaled).  bf16, groups = 1.
cudaError_t launch_reparam_dgrad(const Problem &pb, const void *w, const float *s_vec, void *w_t,
                                 cudaStream_t st);
// One parity class of a strided backward-data pass: w_t[ci][mh][mw][co] = s[co] w[co][r][q][ci] with
// r = r_max - step_h mh, q = q_max - step_w mw for mh < th, mw < tw.
// Per-tap placement for launch_reparam_dgrad_classes (strided backward data, at most 64 taps).
struct ClassTapTable {
    long long offset[64];   // element offset of the tap's class matrix in the scratch buffer
    int count[64];          // taps of that class (0: unused tap)
    int pos[64];            // position of the tap inside its class, row-major over (tap row, tap column)
};
cudaError_t launch_reparam_dgrad_classes(const Problem &pb, const void *w, const float *s_vec, void *w_t,
                                         const ClassTapTable &where, cudaStream_t st);
cudaError_t launch_reparam_dgrad_class(const Problem &pb, const void *w, const float *s_vec, void *w_t, int th,
                                       int tw, int r_max, int q_max, int step_h, int step_w, cudaStream_t st);

// ---- tensor-core weight gradient (bf16 NHWC, groups = 1, channels multiples of 64) ---------------
struct UmmaWgradPlan {
    int splits = 1;           // pixel slices = partial tiles
    long long per_split = 0;  // pixels per slice
    int kt = 1;               // k ranges of the epilogue (rows of dotpart)
    int kr = 8;               // k rows per epilogue block (8 or 2)
};
bool umma_wgrad_eligible(const Problem &pb);
UmmaWgradPlan umma_wgrad_plan(const Problem &pb);
// partials: [splits][kdim][C_out] fp32 (k-major: the transpose of the weight layout)
// bsum    : [splits][C_out] fp32 per-slice sums of dZ over pixels (from a ones row in the GEMM)
// counters: C_out / 32 words zeroed for the fused epilogue (may be NULL)
cudaError_t launch_umma_wgrad(const Problem &pb, const UmmaWgradPlan &pl, const void *dz, const void *x,
                              float *partials, float *bsum, unsigned int *counters, cudaStream_t st);
// Everything after the GEMM in one kernel: dw[co][k] = scale[co] * sum_splits partials (scale = first
// C_out floats of vec3, 1 if NULL); with need_sums also dbeta, db, dgamma (vec3 given) or db = sum dZ.
// dotpart: [kt][C_out] scratch; counters: C_out / 32 zeroed words.
cudaError_t launch_wgrad_epilogue_fused(const Problem &pb, const UmmaWgradPlan &pl, const float *partials,
                                        const float *bsum, const void *w, const float *vec3, const float *b,
                                        const float *mean, float *dw, float *dotpart, unsigned int *counters,
                                        float *db, float *dgamma, float *dbeta, bool need_sums, cudaStream_t st);

// ---- first-layer convolutions with C_in <= 8 (see stem_kernels.cu) -------------------------------
bool stem_eligible(const Problem &pb);
void stem_geometry(const Problem &pb, int *hp, int *wp);     // extent of the packed, zero-bordered input (packed pixels)
bool stem_s2d(const Problem &pb);                            // stride 2, C_in <= 4: 2 x 2 pixel blocks per packed pixel
bool stem_ones_in_pack(const Problem &pb);                   // the packed input carries a constant-1 slot (sum dZ row 3)
int stem_krows(const Problem &pb);                           // 64-wide K rows per output pixel: kh, or ceil(kh / 2)
// byte strides of the 5-D window view {64, w_out, h_out, krows, n} of the packed input
void stem_window_strides(const Problem &pb, unsigned long long str[5]);
size_t stem_packed_bytes(const Problem &pb);                 // [n][hp][wp][8] bf16, or [n][hp][wp][2][2][4]
size_t stem_weight_bytes(const Problem &pb);                 // [C_out][krows][64] bf16
cudaError_t launch_stem_pack(const Problem &pb, const void *x, void *x_packed, cudaStream_t st);
cudaError_t launch_stem_expand_weights(const Problem &pb, const void *w, const float *s_vec, void *wst,
                                       cudaStream_t st);
// Backward data of a stem layer on warp-level MMAs (m16n8k16, fp32 accumulation; the scale is folded into
// the weight fragments it stages).  Used for the narrow-input shapes the sub-pixel GEMM does not take.
bool stem_dgrad_eligible(const Problem &pb);
cudaError_t launch_stem_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                              cudaStream_t st);
// Weight gradient of a stem layer on the packed input: partials [splits][krows * 64][C_out] (padded k rows),
// bsum [splits][C_out]; the epilogue gathers the real kh x kw x C_in entries.
UmmaWgradPlan stem_wgrad_plan(const Problem &pb);
cudaError_t launch_stem_wgrad(const Problem &pb, const UmmaWgradPlan &pl, const void *dz, const void *x_packed,
                              float *partials, float *bsum, cudaStream_t st);
cudaError_t launch_wgrad_epilogue_stem(const Problem &pb, const UmmaWgradPlan &pl, const float *partials,
                                       const float *bsum, const void *w, const float *vec3, const float *b,
                                       const float *mean, float *dw, float *db, float *dgamma, float *dbeta,
                                       bool need_sums, cudaStream_t st);
// Forward pass straight from X for stride_w = 2, C_in <= 4, C_out 64 or 128 (see stem_window.cu): input rows
// staged once in shared memory, the im2col windows formed by the MMA operand addressing.  No packed copy.
bool stem_window_eligible(const Problem &pb);
cudaError_t launch_stem_window_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                                   cudaStream_t st, const BnFold *fold = nullptr);
// Weight gradient of the same layers (C_in <= 3, C_out = 64) straight from X and dZ: one fp32 partial
// [kdim][C_out] and one row of sums of dZ per CTA (stem_window_wgrad_ctas of them), in the layout the fused
// epilogue of the dense weight-gradient path reads; `counters` are zeroed for it.
bool stem_window_wgrad_eligible(const Problem &pb);
int stem_window_wgrad_ctas(const Problem &pb);
cudaError_t launch_stem_window_wgrad(const Problem &pb, const void *dz, const void *x, float *partials, float *bsum,
                                     unsigned int *counters, cudaStream_t st);
// Backward data of the same layers (C_out = 64, W_out <= 128) as a scatter GEMM with the overlap-add of the
// window positions done on chip (see stem_window_dgrad.cu); s_vec (NULL = 1) is folded into the weights.
bool stem_window_dgrad_eligible(const Problem &pb);
cudaError_t launch_stem_window_dgrad(const Problem &pb, const void *dz, const void *w, const float *s_vec, void *dx,
                                     cudaStream_t st);
// k rows per block (kr) and row blocks (kt) of the fused epilogue for pl.splits partial tiles
void wgrad_epilogue_shape(const Problem &pb, UmmaWgradPlan *pl);
cudaError_t launch_stem_fwd(const Problem &pb, const void *x_packed, const void *wst, const float *bias, void *out,
                            cudaStream_t st, const BnFold *fold = nullptr);

// ---- depthwise (groups = C_in = C_out) bandwidth kernels, bf16 NHWC, C multiple of 8 -----------
bool dw_eligible(const Problem &pb);
// 3x3, unit stride and dilation, C <= 256: TMA-fed streaming kernel (forward; backward data with rotated taps)
bool dw_tma_eligible(const Problem &pb);
cudaError_t launch_dw_tma(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                          cudaStream_t st, const BnFold *fold = nullptr, const float *scale = nullptr,
                          bool reverse_taps = false);
// backward weight on the same stream: block partials [nparts][C][10] (9 taps, then sum dZ), then the finish
size_t dw_tma_wgrad_partial_bytes(const Problem &pb);
cudaError_t launch_dw_tma_wgrad(const Problem &pb, const void *dz, const void *x, float *part, int *nparts,
                                cudaStream_t st);
cudaError_t launch_dw_wgrad_finish(const Problem &pb, const float *part, int nparts, const void *w, const float *vec3,
                                   const float *b, const float *mean, float *dw, float *db, float *dgamma,
                                   float *dbeta, cudaStream_t st);
bool dw_wgrad_supported(const Problem &pb);     // tap counts the register-tiled kernel is built for
cudaError_t launch_dw_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                          cudaStream_t st);
cudaError_t launch_dw_dgrad(const Problem &pb, const void *dz, const void *w, void *dx, cudaStream_t st);
int dw_wgrad_splits(const Problem &pb);
// part: [splits][C][taps] fp32 (the layout of the direct weight-gradient partials)
cudaError_t launch_dw_wgrad(const Problem &pb, const void *dz, const void *x, float *part, int splits,
                            cudaStream_t st);

// ---- grouped convolution on the tensor cores as a block-diagonal GEMM ----------------------------
// For C_in/G = C_out/G = cg dividing 64 and C a multiple of 64, every 64-channel block is a dense
// 64 -> 64 convolution whose weight matrix is zero outside the cg x cg diagonal blocks.
bool grouped_bd_eligible(const Problem &pb);
// 8 channels per group, unit stride and dilation, at most 10 taps: warp-level MMAs fed by a TMA patch ring
bool grouped8_eligible(const Problem &pb);
cudaError_t launch_grouped8_fwd(const Problem &pb, const void *x, const void *w, const float *bias, void *z,
                                cudaStream_t st);
cudaError_t launch_grouped8_flip_weights(const Problem &pb, const void *w, const float *s_vec, void *wt,
                                         cudaStream_t st);
cudaError_t launch_grouped8_dgrad(const Problem &pb, const void *dz, const void *wt, void *dx, cudaStream_t st);
// backward weight: part [slots][C][taps 8] and bsum [slots][C] floats, slots = grouped8_wgrad_slots(pb)
int grouped8_wgrad_slots(const Problem &pb);
cudaError_t launch_grouped8_wgrad(const Problem &pb, const void *dz, const void *x, float *part, float *bsum,
                                  cudaStream_t st);
cudaError_t launch_grouped8_wgrad_finish(const Problem &pb, const float *part, const float *bsum, const void *w,
                                         const float *vec3, const float *b, const float *mean, float *dw, float *db,
                                         float *dgamma, float *dbeta, cudaStream_t st);
// wbd[co][tap][64]: omega (scaled by s_vec[co] if given) placed at its group's columns, zeros elsewhere.
// transpose_flip = true builds the backward-data operand instead: wbd[ci][taps-1-tap][64 output channels].
cudaError_t launch_expand_blockdiag(const Problem &pb, const void *w, const float *s_vec, void *wbd,
                                    bool transpose_flip, cudaStream_t st);
// Parameter-gradient epilogue over block-diagonal partials part[split][block][tap * 64 + ci][64 co]:
// same outputs as launch_wgrad_epilogue.
cudaError_t launch_wgrad_epilogue_bd(const Problem &pb, const float *partials, int splits,
                                     const float *bsum_part, int bsplits, const void *w, const float *vec3,
                                     const float *b, const float *mean, float *dw, float *db, float *dgamma,
                                     float *dbeta, cudaStream_t st);

// ---- per-channel reductions (Appendix B: backward of a broadcast is a sum) -------------------
int channel_sum_splits(const Problem &pb);
// part: [splits][C_out] partial sums of t over pixel slices
cudaError_t launch_channel_sum_partial(const Problem &pb, int dtype, int layout, const void *t,
                                       float *part, int splits, cudaStream_t st);

// Finishes the parameter gradients from fp32 partials (fixed summation order):
//   dwf = sum_splits partials;  dsum = sum_splits bsum_part
//   tune mode  (vec3 != NULL): dw = s dwf; dbeta = dsum; db = s dsum;
//                              dgamma = r (sum_k dwf w + dsum (b - mean))
//   plain mode (vec3 == NULL): dw = dwf; db = dsum (if db != NULL)
cudaError_t launch_wgrad_epilogue(const Problem &pb, int dtype, const float *partials, int splits,
                                  const float *bsum_part, int bsplits, const void *w,
                                  const float *vec3, const float *b, const float *mean, float *dw,
                                  float *db, float *dgamma, float *dbeta, cudaStream_t st);

// ---- Eval-mode elementwise BatchNorm (Sec. 3.1) ---------------------------------------------
// z = gamma (y - mean) r + beta
cudaError_t launch_bn_eval_fwd(const Problem &pb, int dtype, int layout, const void *y,
                               const float *vec3_eval /* [s | beta - mean s | r] */, void *z,
                               cudaStream_t st);
// dy = s dz; part_g[split][c] = sum dz (y - mean) r; part_b[split][c] = sum dz
cudaError_t launch_bn_eval_bwd(const Problem &pb, int dtype, int layout, const void *dz,
                               const void *y, const float *gamma, const float *mean,
                               const float *var, void *dy, float *part_g, float *part_b,
                               int splits, cudaStream_t st);
// dgamma = sum part_g; dbeta = sum part_b; db = s dbeta (if db != NULL)
cudaError_t launch_bn_eval_finish(const Problem &pb, const float *part_g, const float *part_b,
                                  int splits, const float *gamma, const float *var, float *db,
                                  float *dgamma, float *dbeta, cudaStream_t st);

// ---- fused backward of 1x1 stride-1 layers (see umma_bwd1x1.cu) ----------------------------------------
// dX plus one fp32 partial [C_in][C_out] and one row of sums of dZ per CTA (fused_bwd1x1_ctas of them), in the
// layout the fused epilogue reads; `counters` are zeroed for it.  vec3 = saved [s | b' | r].
bool fused_bwd1x1_eligible(const Problem &pb);
int fused_bwd1x1_ctas(const Problem &pb);
cudaError_t launch_fused_bwd1x1(const Problem &pb, const void *dz, const void *x, const void *w, const float *vec3,
                                void *dx, float *partials, float *bsum, unsigned int *counters, cudaStream_t st);

// ---- elementwise glue between blocks (glue_kernels.cu): mode 0 relu(a), 1 relu(a + b), 2 a masked by b > 0, 3 a + b
cudaError_t launch_glue(int mode, int dtype, const void *a, const void *b, void *out, long long count, cudaStream_t st);

// One block, one bounded wait (limit_ns) on a barrier without arrivals: sets ERRW_TIMEOUT in the error word.
cudaError_t launch_selftest_wait_timeout(unsigned long long limit_ns, cudaStream_t st);

// ---- TransposedConv-BN: pointwise pieces around the convolution kernels (tconv_kernels.cu) ---------------
// Weights [C_in][taps][C_out/G] (nhwc) or [C_in][C_out/G][taps]; the scale belongs to the output channel
// co = (ci / cig) cog + j.
cudaError_t launch_tconv_vec3(int c_out, float eps, const float *b, const float *gamma, const float *beta,
                              const float *mean, const float *var, float *vec3, cudaStream_t st);
cudaError_t launch_tconv_rescale(int dtype, bool nhwc, long long count, int taps, int cig, int cog, const void *w,
                                 const float *s, void *w_out, cudaStream_t st);
cudaError_t launch_tconv_bias(int dtype, bool nhwc, long long count, int c, long long hw, const float *bias, void *z,
                              cudaStream_t st);
// dwp: fp32 domega' in the weight layout; bsum: [bsplits][C_out] partial sums of dZ
cudaError_t launch_tconv_param_epilogue(int dtype, bool nhwc, int c_out, int taps, int cig, int cog, const float *dwp,
                                        const void *w, const float *vec3, const float *b, const float *mean,
                                        const float *bsum, int bsplits, float *dw, float *db, float *dgamma,
                                        float *dbeta, cudaStream_t st);

}  // namespace convbn
