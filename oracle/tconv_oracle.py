"""fp64 numpy oracle of the Tune-mode TransposedConv-BN block.  TEST INFRASTRUCTURE ONLY.

The paper's rewrite applies to any linear layer followed by a frozen BatchNorm (Sec. 3.2.2 states it for the
convolution and the linear layer; the U-Net experiments use transposed convolutions): the per-output-channel
scale commutes with the layer, so

    r = 1 / sqrt(var_hat + eps),  s = gamma r,  omega' = s[co] omega[:, co],  b' = (b - mu_hat) s + beta,
    Z = convT(X, omega') + b'                                                     (Sec. 3.3 definitions)

and the backward pass is Table 2's Tune row with the transposed convolution in place of the convolution.
The transposed convolution is written out as its definition, a scatter: input pixel (hi, wi) adds
X[n, ci, hi, wi] omega[ci, co, r, q] to output pixel (hi stride - pad + r dil, wi stride - pad + q dil).
Weights are [C_in][C_out / G][kh][kw] (the deep-learning convention for transposed convolutions), tensors
logical NCHW.  Loops run over groups and taps only; nothing is blocked, fused or reordered beyond that.

Pinned in tests/test_tconv.py: against the pinned convolution oracle (the transposed convolution is the
adjoint of the convolution with the same weights, so it equals that oracle's conv_grad_input element by
element), against torch.nn.functional.conv_transpose2d, the Eval form (layer, then BatchNorm) and central
finite differences of J = <dZ, Z> for all five gradients.
"""
import numpy as np


def out_hw(h_in, w_in, kh, kw, stride, pad, dil):
    return ((h_in - 1) * stride - 2 * pad + dil * (kh - 1) + 1, (w_in - 1) * stride - 2 * pad + dil * (kw - 1) + 1)


def scale(gamma, var_hat, eps):
    r = 1.0 / np.sqrt(np.asarray(var_hat, dtype=np.float64) + eps)
    return np.asarray(gamma, dtype=np.float64) * r, r


def conv_transpose(x, w, stride=1, pad=0, dil=1, groups=1):
    """The scatter definition.  x [N][C_in][H][W], w [C_in][C_out/G][kh][kw] -> [N][C_out][H_out][W_out]."""
    x, w = np.asarray(x, dtype=np.float64), np.asarray(w, dtype=np.float64)
    n, c_in, h, wd = x.shape
    cog, kh, kw = w.shape[1], w.shape[2], w.shape[3]
    cig = c_in // groups
    ho, wo = out_hw(h, wd, kh, kw, stride, pad, dil)
    full = np.zeros((n, cog * groups, ho + 2 * pad, wo + 2 * pad))          # un-cropped output
    for g in range(groups):
        xg, wg = x[:, g * cig:(g + 1) * cig], w[g * cig:(g + 1) * cig]
        for r in range(kh):
            for q in range(kw):
                contrib = np.einsum("nchw,co->nohw", xg, wg[:, :, r, q])
                full[:, g * cog:(g + 1) * cog, r * dil:r * dil + (h - 1) * stride + 1:stride,
                     q * dil:q * dil + (wd - 1) * stride + 1:stride] += contrib
    return full[:, :, pad:pad + ho, pad:pad + wo]


def _channel_of_weight(c_in, cog, groups):
    """Output channel of weight element [ci][j]: co = (ci // (C_in/G)) (C_out/G) + j, as an index array [C_in][C_out/G]."""
    cig = c_in // groups
    return (np.arange(c_in)[:, None] // cig) * cog + np.arange(cog)[None, :]


def fold(w, b, gamma, beta, mu_hat, var_hat, eps, groups=1):
    s, _ = scale(gamma, var_hat, eps)
    w = np.asarray(w, dtype=np.float64)
    co = _channel_of_weight(w.shape[0], w.shape[1], groups)
    bb = np.zeros_like(s) if b is None else np.asarray(b, dtype=np.float64)
    return w * s[co][:, :, None, None], (bb - np.asarray(mu_hat, dtype=np.float64)) * s + np.asarray(beta, dtype=np.float64)


def tune_forward(x, w, b, gamma, beta, mu_hat, var_hat, eps, stride=1, pad=0, dil=1, groups=1):
    w_f, b_f = fold(w, b, gamma, beta, mu_hat, var_hat, eps, groups)
    z = conv_transpose(x, w_f, stride, pad, dil, groups) + b_f[None, :, None, None]
    return {"z": z, "w_f": w_f, "b_f": b_f}


def eval_forward(x, w, b, gamma, beta, mu_hat, var_hat, eps, stride=1, pad=0, dil=1, groups=1):
    """Layer, then BatchNorm with the running statistics (Sec. 3.1)."""
    y = conv_transpose(x, w, stride, pad, dil, groups)
    if b is not None:
        y = y + np.asarray(b, dtype=np.float64)[None, :, None, None]
    s, _ = scale(gamma, var_hat, eps)
    bc = lambda v: np.asarray(v, dtype=np.float64)[None, :, None, None]
    return (y - bc(mu_hat)) * s[None, :, None, None] + bc(beta)


def tune_backward(dz, x, w, b, gamma, mu_hat, var_hat, eps, stride=1, pad=0, dil=1, groups=1):
    """Table 2, Tune row, for the transposed convolution: gradients of J with dJ/dZ = dz."""
    dz, x, w = (np.asarray(t, dtype=np.float64) for t in (dz, x, w))
    n, c_in, h, wd = x.shape
    cog, kh, kw = w.shape[1], w.shape[2], w.shape[3]
    cig = c_in // groups
    s, r = scale(gamma, var_hat, eps)
    co = _channel_of_weight(c_in, cog, groups)
    w_f = w * s[co][:, :, None, None]
    dzp = np.pad(dz, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    dx, dw_f = np.zeros_like(x), np.zeros_like(w)
    for g in range(groups):
        for rr in range(kh):
            for q in range(kw):
                # the output pixels input pixel (hi, wi) scattered to through tap (rr, q)
                win = dzp[:, g * cog:(g + 1) * cog, rr * dil:rr * dil + (h - 1) * stride + 1:stride,
                          q * dil:q * dil + (wd - 1) * stride + 1:stride]
                dx[:, g * cig:(g + 1) * cig] += np.einsum("nohw,co->nchw", win, w_f[g * cig:(g + 1) * cig, :, rr, q])
                dw_f[g * cig:(g + 1) * cig, :, rr, q] = np.einsum("nchw,nohw->co", x[:, g * cig:(g + 1) * cig], win)
    dbeta = dz.sum(axis=(0, 2, 3))
    bb = np.zeros_like(s) if b is None else np.asarray(b, dtype=np.float64)
    dot = np.zeros_like(s)
    np.add.at(dot, co, (dw_f * w).sum(axis=(2, 3)))          # sum over C_in/G, kh, kw of domega' omega, per output channel
    return {"dx": dx, "dw": dw_f * s[co][:, :, None, None], "db": None if b is None else s * dbeta,
            "dgamma": r * (dot + dbeta * (bb - np.asarray(mu_hat, dtype=np.float64))), "dbeta": dbeta, "dw_f": dw_f}
