"""numpy front end of the fp64 CPU oracle (``convbn_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the CPU-baseline timing import this;
the CUDA library and its Python binding never do, and this module imports neither.

All arrays are float64, C-contiguous, in the paper's logical order (Sec. 3.1, Appendix C):
``x [N, C_in, H_in, W_in]``, ``w [C_out, C_in/G, kh, kw]``, per-channel vectors ``[C_out]``,
``y / z / dz [N, C_out, H_out, W_out]``.
"""
import ctypes
from dataclasses import dataclass

import numpy as np

from . import build as _build


class _CShape(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int) for k in (
        "n", "c_in", "h_in", "w_in", "c_out", "kh", "kw", "stride_h", "stride_w",
        "pad_h", "pad_w", "dil_h", "dil_w", "groups")] + [("eps", ctypes.c_double)]


@dataclass(frozen=True)
class Shape:
    """Problem size of one ConvBN block (Sec. 3.1), with the conv hyper-parameters the paper
    leaves implicit spelled out."""
    n: int
    c_in: int
    h_in: int
    w_in: int
    c_out: int
    kh: int
    kw: int
    stride_h: int = 1
    stride_w: int = 1
    pad_h: int = 0
    pad_w: int = 0
    dil_h: int = 1
    dil_w: int = 1
    groups: int = 1
    eps: float = 1e-5

    def c(self) -> _CShape:
        return _CShape(self.n, self.c_in, self.h_in, self.w_in, self.c_out, self.kh, self.kw,
                       self.stride_h, self.stride_w, self.pad_h, self.pad_w, self.dil_h,
                       self.dil_w, self.groups, float(self.eps))

    @property
    def x_shape(self):
        return (self.n, self.c_in, self.h_in, self.w_in)

    @property
    def w_shape(self):
        return (self.c_out, self.c_in // self.groups, self.kh, self.kw)

    @property
    def z_shape(self):
        ho, wo = out_hw(self)
        return (self.n, self.c_out, ho, wo)


_lib = None
_DP = ctypes.POINTER(ctypes.c_double)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_out_hw.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(t: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(int(t)))


def _p(a):
    if a is None:
        return ctypes.cast(None, _DP)
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_DP)


def _f64(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def out_hw(s: Shape):
    ho, wo = ctypes.c_int(0), ctypes.c_int(0)
    cs = s.c()
    if lib().oracle_out_hw(ctypes.byref(cs), ctypes.byref(ho), ctypes.byref(wo)) != 0:
        raise ValueError("invalid convolution shape: %r" % (s,))
    return ho.value, wo.value


def scale(s: Shape, gamma, var_hat):
    """(s, r) with s = gamma / sqrt(var_hat + eps), r = 1 / sqrt(var_hat + eps)."""
    cs = s.c()
    sc, r = np.empty(s.c_out), np.empty(s.c_out)
    lib().oracle_scale(ctypes.byref(cs), _p(_f64(gamma, (s.c_out,))),
                       _p(_f64(var_hat, (s.c_out,))), _p(sc), _p(r))
    return sc, r


def conv(s: Shape, x, w, b=None):
    cs = s.c()
    x, w, b = _f64(x, s.x_shape), _f64(w, s.w_shape), _f64(b, (s.c_out,))
    y = np.empty(s.z_shape)
    lib().oracle_conv(ctypes.byref(cs), _p(x), _p(w), _p(b), _p(y))
    return y


def bn_eval(s: Shape, y, gamma, beta, mu_hat, var_hat):
    cs = s.c()
    y = _f64(y, s.z_shape)
    z = np.empty_like(y)
    v = [_f64(t, (s.c_out,)) for t in (gamma, beta, mu_hat, var_hat)]
    lib().oracle_bn_eval(ctypes.byref(cs), _p(y), _p(v[0]), _p(v[1]), _p(v[2]), _p(v[3]), _p(z))
    return z


def fold(s: Shape, w, b, gamma, beta, mu_hat, var_hat):
    """(omega', b') of Sec. 3.3."""
    cs = s.c()
    w, b = _f64(w, s.w_shape), _f64(b, (s.c_out,))
    v = [_f64(t, (s.c_out,)) for t in (gamma, beta, mu_hat, var_hat)]
    w_f, b_f = np.empty(s.w_shape), np.empty(s.c_out)
    lib().oracle_fold(ctypes.byref(cs), _p(w), _p(b), _p(v[0]), _p(v[1]), _p(v[2]), _p(v[3]),
                      _p(w_f), _p(b_f))
    return w_f, b_f


def sum_per_channel(s: Shape, t):
    cs = s.c()
    t = _f64(t, s.z_shape)
    out = np.empty(s.c_out)
    lib().oracle_sum_per_channel(ctypes.byref(cs), _p(t), _p(out))
    return out


def conv_grad_weight(s: Shape, dy, x):
    cs = s.c()
    dy, x = _f64(dy, s.z_shape), _f64(x, s.x_shape)
    dw = np.empty(s.w_shape)
    lib().oracle_conv_grad_weight(ctypes.byref(cs), _p(dy), _p(x), _p(dw))
    return dw


def conv_grad_input(s: Shape, dy, w):
    cs = s.c()
    dy, w = _f64(dy, s.z_shape), _f64(w, s.w_shape)
    dx = np.empty(s.x_shape)
    lib().oracle_conv_grad_input(ctypes.byref(cs), _p(dy), _p(w), _p(dx))
    return dx


def eval_forward(s: Shape, x, w, b, gamma, beta, mu_hat, var_hat):
    """Eval mode: returns dict(y=..., z=...); y is what Eval mode saves for backward."""
    cs = s.c()
    x, w, b = _f64(x, s.x_shape), _f64(w, s.w_shape), _f64(b, (s.c_out,))
    v = [_f64(t, (s.c_out,)) for t in (gamma, beta, mu_hat, var_hat)]
    y, z = np.empty(s.z_shape), np.empty(s.z_shape)
    lib().oracle_eval_forward(ctypes.byref(cs), _p(x), _p(w), _p(b), _p(v[0]), _p(v[1]),
                              _p(v[2]), _p(v[3]), _p(y), _p(z))
    return {"y": y, "z": z}


def eval_backward(s: Shape, dz, x, y, w, gamma, mu_hat, var_hat, with_bias=True):
    cs = s.c()
    dz, x, y, w = _f64(dz, s.z_shape), _f64(x, s.x_shape), _f64(y, s.z_shape), _f64(w, s.w_shape)
    v = [_f64(t, (s.c_out,)) for t in (gamma, mu_hat, var_hat)]
    dx, dw = np.empty(s.x_shape), np.empty(s.w_shape)
    db = np.empty(s.c_out) if with_bias else None
    dg, dbt = np.empty(s.c_out), np.empty(s.c_out)
    lib().oracle_eval_backward(ctypes.byref(cs), _p(dz), _p(x), _p(y), _p(w), _p(v[0]),
                               _p(v[1]), _p(v[2]), _p(dx), _p(dw), _p(db), _p(dg), _p(dbt))
    return {"dx": dx, "dw": dw, "db": db, "dgamma": dg, "dbeta": dbt}


def deploy_forward(s: Shape, x, w_f, b_f):
    return conv(s, x, w_f, b_f)


def deploy_backward(s: Shape, dz, x, w_f):
    cs = s.c()
    dz, x, w_f = _f64(dz, s.z_shape), _f64(x, s.x_shape), _f64(w_f, s.w_shape)
    dx, dw_f, db_f = np.empty(s.x_shape), np.empty(s.w_shape), np.empty(s.c_out)
    lib().oracle_deploy_backward(ctypes.byref(cs), _p(dz), _p(x), _p(w_f), _p(dx), _p(dw_f),
                                 _p(db_f))
    return {"dx": dx, "dw_f": dw_f, "db_f": db_f}


def tune_forward(s: Shape, x, w, b, gamma, beta, mu_hat, var_hat):
    """Tune mode forward: dict(z, w_f, b_f); w_f (omega') is what Tune keeps beside x."""
    cs = s.c()
    x, w, b = _f64(x, s.x_shape), _f64(w, s.w_shape), _f64(b, (s.c_out,))
    v = [_f64(t, (s.c_out,)) for t in (gamma, beta, mu_hat, var_hat)]
    w_f, b_f, z = np.empty(s.w_shape), np.empty(s.c_out), np.empty(s.z_shape)
    lib().oracle_tune_forward(ctypes.byref(cs), _p(x), _p(w), _p(b), _p(v[0]), _p(v[1]),
                              _p(v[2]), _p(v[3]), _p(w_f), _p(b_f), _p(z))
    return {"z": z, "w_f": w_f, "b_f": b_f}


def tune_backward(s: Shape, dz, x, w, w_f, b, gamma, mu_hat, var_hat):
    cs = s.c()
    dz, x = _f64(dz, s.z_shape), _f64(x, s.x_shape)
    w, w_f, b = _f64(w, s.w_shape), _f64(w_f, s.w_shape), _f64(b, (s.c_out,))
    v = [_f64(t, (s.c_out,)) for t in (gamma, mu_hat, var_hat)]
    dx, dw = np.empty(s.x_shape), np.empty(s.w_shape)
    db = np.empty(s.c_out) if b is not None else None
    dg, dbt = np.empty(s.c_out), np.empty(s.c_out)
    lib().oracle_tune_backward(ctypes.byref(cs), _p(dz), _p(x), _p(w), _p(w_f), _p(b), _p(v[0]),
                               _p(v[1]), _p(v[2]), _p(dx), _p(dw), _p(db), _p(dg), _p(dbt))
    return {"dx": dx, "dw": dw, "db": db, "dgamma": dg, "dbeta": dbt}


def saved_elements(s: Shape, mode: str) -> int:
    """Elements kept for the backward pass per block (Sec. 3.3, Sec. 3.4, Appendix M memory
    analysis): Eval X + Y, Deploy X, Tune X + omega'."""
    ho, wo = out_hw(s)
    x = s.n * s.c_in * s.h_in * s.w_in
    y = s.n * s.c_out * ho * wo
    wf = s.c_out * (s.c_in // s.groups) * s.kh * s.kw
    return {"eval": x + y, "deploy": x, "tune": x + wf}[mode]


def rel_l2(got, ref) -> float:
    """||got - ref||_2 / ||ref||_2 in fp64 (absolute norm of got if ref is identically 0)."""
    got = np.asarray(got, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    assert got.shape == ref.shape, (got.shape, ref.shape)
    den = float(np.linalg.norm(ref))
    num = float(np.linalg.norm(got - ref))
    return num if den == 0.0 else num / den
