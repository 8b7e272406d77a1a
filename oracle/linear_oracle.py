"""Plain fp64 definition of a Linear-BN block in Tune mode (test infrastructure, numpy only).

Sec. 3.2.2 notes that the per-channel scale commutes with a linear layer as it does with a convolution, so the
Tune-mode block of Sec. 3.4 and the Tune row of Table 2 carry over with the convolution replaced by a matrix
product: X [rows, in], W [out, in], b / gamma / beta / mu_hat / var_hat [out].

    r = 1 / sqrt(var_hat + eps)   s = gamma r   W' = s W (rows scaled)   b' = (b - mu_hat) s + beta
    Z = X W'^T + b'
    dX = dZ W'      dW' = dZ^T X      dW = s dW'      dbeta = sum_rows dZ      db = s dbeta
    dgamma = r (sum_in dW' W + dbeta (b - mu_hat))

Only tests/, the smoke entry and the benchmark's CPU baseline may import this module; the CUDA path never does.
"""
import numpy as np


def tune_forward(x, w, b, gamma, beta, mu_hat, var_hat, eps):
    x, w = np.asarray(x, np.float64), np.asarray(w, np.float64)
    r = 1.0 / np.sqrt(np.asarray(var_hat, np.float64) + eps)
    s = np.asarray(gamma, np.float64) * r
    b0 = np.zeros(w.shape[0]) if b is None else np.asarray(b, np.float64)
    w_f = s[:, None] * w
    b_f = (b0 - np.asarray(mu_hat, np.float64)) * s + np.asarray(beta, np.float64)
    return {"z": x @ w_f.T + b_f[None, :], "w_f": w_f, "b_f": b_f, "s": s, "r": r}


def tune_backward(dz, x, w, b, gamma, mu_hat, var_hat, eps):
    dz, x, w = np.asarray(dz, np.float64), np.asarray(x, np.float64), np.asarray(w, np.float64)
    r = 1.0 / np.sqrt(np.asarray(var_hat, np.float64) + eps)
    s = np.asarray(gamma, np.float64) * r
    b0 = np.zeros(w.shape[0]) if b is None else np.asarray(b, np.float64)
    dw_f = dz.T @ x
    dbeta = dz.sum(axis=0)
    out = {"dx": dz @ (s[:, None] * w), "dw": s[:, None] * dw_f, "dbeta": dbeta,
           "dgamma": r * ((dw_f * w).sum(axis=1) + dbeta * (b0 - np.asarray(mu_hat, np.float64))),
           "db": None if b is None else s * dbeta}
    return out


def eval_forward(x, w, b, gamma, beta, mu_hat, var_hat, eps):
    """Sec. 3.1 Eval form: the linear layer, then BatchNorm with the tracked statistics."""
    x, w = np.asarray(x, np.float64), np.asarray(w, np.float64)
    y = x @ w.T + (0.0 if b is None else np.asarray(b, np.float64)[None, :])
    return np.asarray(gamma)[None, :] * (y - np.asarray(mu_hat)[None, :]) / np.sqrt(np.asarray(var_hat)[None, :] + eps) + \
        np.asarray(beta)[None, :]
