/*
 * fp64 CPU oracle for Convolution-BatchNorm blocks in Eval, Deploy and Tune mode.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * library is checked against.  It shares no code, header, table or helper with the
 * CUDA path, and nothing on the product path may call it.
 *
 * Everything is double precision, tensors are dense and in the paper's logical order
 * (Sec. 3.1, Appendix C shape annotations):
 *     X  [N][C_in][H_in][W_in]        omega [C_out][C_in/G][kh][kw]
 *     Y,Z,dZ [N][C_out][H_out][W_out] b, gamma, beta, mu_hat, var_hat [C_out]
 * The paper writes only a kernel size k; stride, padding, dilation and groups follow
 * the usual deep-learning convention: zero padding, floor output size, cross-correlation
 * in the forward pass (the paper's "omega_rot" appears in the backward pass only),
 * contiguous channel groups.  The BatchNorm buffer holds the running VARIANCE and eps is
 * added under the root (all of the paper's formulas use sqrt(var_hat + eps)).
 *
 * Parity status: every function here is pinned by tests that do not go through this
 * file's own formulas (finite differences of J = <dZ, Z>, adjoint identities, library
 * correlation / matmul special cases, brute-force group/stride/dilation constructions,
 * closed forms).  Nothing is "parity unpinned".
 *
 * Loops are direct (no im2col, no GEMM, no blocking).  OpenMP only distributes disjoint
 * output slices over threads; the arithmetic order inside a slice is the loop order.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int n, c_in, h_in, w_in, c_out, kh, kw;
    int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, groups;
    double eps;
} oracle_shape;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* Output extent: floor((in + 2 pad - dil (k-1) - 1) / stride) + 1.  Returns 0 on success. */
int oracle_out_hw(const oracle_shape *s, int *h_out, int *w_out) {
    if (!s || s->n <= 0 || s->c_in <= 0 || s->c_out <= 0 || s->kh <= 0 || s->kw <= 0 ||
        s->stride_h <= 0 || s->stride_w <= 0 || s->dil_h <= 0 || s->dil_w <= 0 ||
        s->pad_h < 0 || s->pad_w < 0 || s->groups <= 0 || s->c_in % s->groups ||
        s->c_out % s->groups)
        return 1;
    int eh = s->h_in + 2 * s->pad_h - s->dil_h * (s->kh - 1) - 1;
    int ew = s->w_in + 2 * s->pad_w - s->dil_w * (s->kw - 1) - 1;
    if (eh < 0 || ew < 0) return 1;
    *h_out = eh / s->stride_h + 1;
    *w_out = ew / s->stride_w + 1;
    return 0;
}

/* s = gamma / sqrt(var_hat + eps),  r = 1 / sqrt(var_hat + eps)   (Sec. 3.3 definitions) */
void oracle_scale(const oracle_shape *sh, const double *gamma, const double *var_hat,
                  double *s, double *r) {
    for (int co = 0; co < sh->c_out; ++co) {
        double inv = 1.0 / sqrt(var_hat[co] + sh->eps);
        if (r) r[co] = inv;
        if (s) s[co] = gamma[co] * inv;
    }
}

/* Y = omega (*) X + b   (Sec. 3.1; cross-correlation, zero padding).  b may be NULL. */
void oracle_conv(const oracle_shape *s, const double *x, const double *w, const double *b,
                 double *y) {
    int ho_n, wo_n;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return;
    const int cg = s->c_in / s->groups, cog = s->c_out / s->groups;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < s->n; ++n)
        for (int co = 0; co < s->c_out; ++co) {
            const int g = co / cog;
            double *yp = y + ((size_t)n * s->c_out + co) * ho_n * wo_n;
            const double b0 = b ? b[co] : 0.0;
            for (int i = 0; i < ho_n * wo_n; ++i) yp[i] = b0;
            for (int ci = 0; ci < cg; ++ci) {
                const double *xp = x + ((size_t)n * s->c_in + g * cg + ci) * s->h_in * s->w_in;
                for (int r = 0; r < s->kh; ++r)
                    for (int q = 0; q < s->kw; ++q) {
                        const double wv = w[(((size_t)co * cg + ci) * s->kh + r) * s->kw + q];
                        for (int ho = 0; ho < ho_n; ++ho) {
                            const int hi = ho * s->stride_h - s->pad_h + r * s->dil_h;
                            if (hi < 0 || hi >= s->h_in) continue;
                            for (int wo = 0; wo < wo_n; ++wo) {
                                const int wi = wo * s->stride_w - s->pad_w + q * s->dil_w;
                                if (wi < 0 || wi >= s->w_in) continue;
                                yp[ho * wo_n + wo] += wv * xp[hi * s->w_in + wi];
                            }
                        }
                    }
            }
        }
}

/* Z = gamma (Y - mu_hat) / sqrt(var_hat + eps) + beta   (Sec. 3.1, Eval mode) */
void oracle_bn_eval(const oracle_shape *s, const double *y, const double *gamma,
                    const double *beta, const double *mu_hat, const double *var_hat,
                    double *z) {
    int ho_n, wo_n;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return;
    const size_t hw = (size_t)ho_n * wo_n;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < s->n; ++n)
        for (int co = 0; co < s->c_out; ++co) {
            const double den = sqrt(var_hat[co] + s->eps);
            const double *yp = y + ((size_t)n * s->c_out + co) * hw;
            double *zp = z + ((size_t)n * s->c_out + co) * hw;
            for (size_t i = 0; i < hw; ++i)
                zp[i] = gamma[co] * ((yp[i] - mu_hat[co]) / den) + beta[co];
        }
}

/* omega' = s . omega (per output channel),  b' = (b - mu_hat) s + beta   (Sec. 3.3) */
void oracle_fold(const oracle_shape *sh, const double *w, const double *b,
                 const double *gamma, const double *beta, const double *mu_hat,
                 const double *var_hat, double *w_f, double *b_f) {
    const size_t k = (size_t)(sh->c_in / sh->groups) * sh->kh * sh->kw;
    for (int co = 0; co < sh->c_out; ++co) {
        const double sc = gamma[co] / sqrt(var_hat[co] + sh->eps);
        for (size_t i = 0; i < k; ++i) w_f[co * k + i] = sc * w[co * k + i];
        b_f[co] = ((b ? b[co] : 0.0) - mu_hat[co]) * sc + beta[co];
    }
}

/* out[co] = sum over N, H_out, W_out of t[n][co][ho][wo]   (Appendix B: the backward of a
 * broadcast is the sum over the broadcast dimensions) */
void oracle_sum_per_channel(const oracle_shape *s, const double *t, double *out) {
    int ho_n, wo_n;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return;
    const size_t hw = (size_t)ho_n * wo_n;
#pragma omp parallel for schedule(static)
    for (int co = 0; co < s->c_out; ++co) {
        double acc = 0.0;
        for (int n = 0; n < s->n; ++n) {
            const double *tp = t + ((size_t)n * s->c_out + co) * hw;
            for (size_t i = 0; i < hw; ++i) acc += tp[i];
        }
        out[co] = acc;
    }
}

/* dJ/domega = dJ/dY (.) X   (Sec. 3.2.1): the cross-correlation of the output gradient with
 * the input, i.e. dw[co][ci][r][q] = sum_{n,ho,wo} dy[n][co][ho][wo] x[n][g Cg+ci][hi][wi]. */
void oracle_conv_grad_weight(const oracle_shape *s, const double *dy, const double *x,
                             double *dw) {
    int ho_n, wo_n;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return;
    const int cg = s->c_in / s->groups, cog = s->c_out / s->groups;
#pragma omp parallel for collapse(2) schedule(static)
    for (int co = 0; co < s->c_out; ++co)
        for (int ci = 0; ci < cg; ++ci) {
            const int g = co / cog;
            for (int r = 0; r < s->kh; ++r)
                for (int q = 0; q < s->kw; ++q) {
                    double acc = 0.0;
                    for (int n = 0; n < s->n; ++n) {
                        const double *dyp = dy + ((size_t)n * s->c_out + co) * ho_n * wo_n;
                        const double *xp =
                            x + ((size_t)n * s->c_in + g * cg + ci) * s->h_in * s->w_in;
                        for (int ho = 0; ho < ho_n; ++ho) {
                            const int hi = ho * s->stride_h - s->pad_h + r * s->dil_h;
                            if (hi < 0 || hi >= s->h_in) continue;
                            for (int wo = 0; wo < wo_n; ++wo) {
                                const int wi = wo * s->stride_w - s->pad_w + q * s->dil_w;
                                if (wi < 0 || wi >= s->w_in) continue;
                                acc += dyp[ho * wo_n + wo] * xp[hi * s->w_in + wi];
                            }
                        }
                    }
                    dw[(((size_t)co * cg + ci) * s->kh + r) * s->kw + q] = acc;
                }
        }
}

/* dJ/dX = omega_rot (*) dJ/dY   (Sec. 3.2.1), written as the literal adjoint of
 * oracle_conv: every (output position, tap) pair that read x[hi][wi] in the forward pass
 * adds w * dy into dx[hi][wi].  One thread owns one (n, input channel) plane. */
void oracle_conv_grad_input(const oracle_shape *s, const double *dy, const double *w,
                            double *dx) {
    int ho_n, wo_n;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return;
    const int cg = s->c_in / s->groups, cog = s->c_out / s->groups;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < s->n; ++n)
        for (int c = 0; c < s->c_in; ++c) {
            const int g = c / cg, ci = c % cg;
            double *dxp = dx + ((size_t)n * s->c_in + c) * s->h_in * s->w_in;
            for (int i = 0; i < s->h_in * s->w_in; ++i) dxp[i] = 0.0;
            for (int co = g * cog; co < (g + 1) * cog; ++co) {
                const double *dyp = dy + ((size_t)n * s->c_out + co) * ho_n * wo_n;
                for (int r = 0; r < s->kh; ++r)
                    for (int q = 0; q < s->kw; ++q) {
                        const double wv = w[(((size_t)co * cg + ci) * s->kh + r) * s->kw + q];
                        for (int ho = 0; ho < ho_n; ++ho) {
                            const int hi = ho * s->stride_h - s->pad_h + r * s->dil_h;
                            if (hi < 0 || hi >= s->h_in) continue;
                            for (int wo = 0; wo < wo_n; ++wo) {
                                const int wi = wo * s->stride_w - s->pad_w + q * s->dil_w;
                                if (wi < 0 || wi >= s->w_in) continue;
                                dxp[hi * s->w_in + wi] += wv * dyp[ho * wo_n + wo];
                            }
                        }
                    }
            }
        }
}

static size_t out_elems(const oracle_shape *s) {
    int ho_n = 0, wo_n = 0;
    if (oracle_out_hw(s, &ho_n, &wo_n)) return 0;
    return (size_t)s->n * s->c_out * ho_n * wo_n;
}
static size_t w_elems(const oracle_shape *s) {
    return (size_t)s->c_out * (s->c_in / s->groups) * s->kh * s->kw;
}

/* ---- Eval mode (Sec. 3.1; Table 2, Eval row) ------------------------------------------ */

/* Forward: Y = omega (*) X + b is kept (it is what Eval mode saves), Z = BN_eval(Y). */
void oracle_eval_forward(const oracle_shape *s, const double *x, const double *w,
                         const double *b, const double *gamma, const double *beta,
                         const double *mu_hat, const double *var_hat, double *y, double *z) {
    oracle_conv(s, x, w, b, y);
    oracle_bn_eval(s, y, gamma, beta, mu_hat, var_hat, z);
}

/* Backward by the Eval-row equations: dY = s dZ; dX = omega_rot (*) dY; domega = dY (.) X;
 * db = sum dY; dgamma = sum dZ (Y - mu_hat) / sqrt(var_hat + eps); dbeta = sum dZ.
 * db may be NULL. */
void oracle_eval_backward(const oracle_shape *sh, const double *dz, const double *x,
                          const double *y, const double *w, const double *gamma,
                          const double *mu_hat, const double *var_hat, double *dx, double *dw,
                          double *db, double *dgamma, double *dbeta) {
    int ho_n, wo_n;
    if (oracle_out_hw(sh, &ho_n, &wo_n)) return;
    const size_t hw = (size_t)ho_n * wo_n, ne = out_elems(sh);
    double *dy = (double *)malloc(ne * sizeof(double));
    double *t = (double *)malloc(ne * sizeof(double));
    if (!dy || !t) { free(dy); free(t); return; }
    for (int n = 0; n < sh->n; ++n)
        for (int co = 0; co < sh->c_out; ++co) {
            const double den = sqrt(var_hat[co] + sh->eps);
            const double sc = gamma[co] / den;
            const size_t o = ((size_t)n * sh->c_out + co) * hw;
            for (size_t i = 0; i < hw; ++i) {
                dy[o + i] = sc * dz[o + i];
                t[o + i] = dz[o + i] * ((y[o + i] - mu_hat[co]) / den);
            }
        }
    oracle_conv_grad_input(sh, dy, w, dx);
    oracle_conv_grad_weight(sh, dy, x, dw);
    if (db) oracle_sum_per_channel(sh, dy, db);
    oracle_sum_per_channel(sh, t, dgamma);
    oracle_sum_per_channel(sh, dz, dbeta);
    free(dy);
    free(t);
}

/* ---- Deploy mode (Sec. 3.3; Table 2, Deploy row) -------------------------------------- */

void oracle_deploy_forward(const oracle_shape *s, const double *x, const double *w_f,
                           const double *b_f, double *z) {
    oracle_conv(s, x, w_f, b_f, z);
}

/* dX = omega'_rot (*) dZ; domega' = dZ (.) X; db' = sum dZ */
void oracle_deploy_backward(const oracle_shape *s, const double *dz, const double *x,
                            const double *w_f, double *dx, double *dw_f, double *db_f) {
    oracle_conv_grad_input(s, dz, w_f, dx);
    oracle_conv_grad_weight(s, dz, x, dw_f);
    oracle_sum_per_channel(s, dz, db_f);
}

/* ---- Tune mode (Sec. 3.4; Table 2, Tune row) ------------------------------------------ */

/* Forward: omega', b' formed from the current parameters at every call, then one
 * convolution.  No pre-normalisation tensor Y exists.  w_f (omega') is returned because it
 * is what Tune mode keeps for the backward pass beside X. */
void oracle_tune_forward(const oracle_shape *s, const double *x, const double *w,
                         const double *b, const double *gamma, const double *beta,
                         const double *mu_hat, const double *var_hat, double *w_f,
                         double *b_f, double *z) {
    oracle_fold(s, w, b, gamma, beta, mu_hat, var_hat, w_f, b_f);
    oracle_conv(s, x, w_f, b_f, z);
}

/* Backward by the Tune-row equations:
 *   dX      = omega'_rot (*) dZ
 *   domega' = dZ (.) X
 *   domega  = s domega'
 *   dbeta   = sum dZ
 *   db      = s dbeta
 *   dgamma  = ( sum_{ci,r,q} domega' omega  +  dbeta (b - mu_hat) ) / sqrt(var_hat + eps)
 * (the sums the paper leaves implicit are those of Appendix B).  b and db may be NULL. */
void oracle_tune_backward(const oracle_shape *sh, const double *dz, const double *x,
                          const double *w, const double *w_f, const double *b,
                          const double *gamma, const double *mu_hat, const double *var_hat,
                          double *dx, double *dw, double *db, double *dgamma, double *dbeta) {
    const size_t k = (size_t)(sh->c_in / sh->groups) * sh->kh * sh->kw;
    double *dw_f = (double *)malloc(w_elems(sh) * sizeof(double));
    if (!dw_f) return;
    oracle_conv_grad_input(sh, dz, w_f, dx);
    oracle_conv_grad_weight(sh, dz, x, dw_f);
    oracle_sum_per_channel(sh, dz, dbeta);
    for (int co = 0; co < sh->c_out; ++co) {
        const double den = sqrt(var_hat[co] + sh->eps);
        const double sc = gamma[co] / den;
        double dot = 0.0;
        for (size_t i = 0; i < k; ++i) {
            dw[co * k + i] = sc * dw_f[co * k + i];
            dot += dw_f[co * k + i] * w[co * k + i];
        }
        if (db) db[co] = sc * dbeta[co];
        dgamma[co] = dot / den + dbeta[co] * (((b ? b[co] : 0.0) - mu_hat[co]) / den);
    }
    free(dw_f);
}
