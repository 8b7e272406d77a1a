"""Thin ctypes binding of ``libconvbn.so`` (declared in ``include/convbn.h``).

Argument marshalling only: every function has the name and argument order of its C entry point,
takes torch CUDA tensors (or raw integer device addresses, or None for NULL) and returns nothing;
a non-zero status raises ``ConvBNError``.  There is no fallback: if the compiled library is
missing, importing succeeds but the first call raises.
"""
import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIBRARY = os.path.join(_HERE, "libconvbn.so")

OK, EINVAL, EUNSUPPORTED, EWORKSPACE, EALIGN, ECUDA, ETIMEOUT, ECAPACITY = range(8)
F32, BF16, F16 = 0, 1, 2
NCHW, NHWC = 0, 1
MODE_TUNE, MODE_EVAL, MODE_DEPLOY = 0, 1, 2
(PHASE_TUNE_FWD, PHASE_TUNE_BWD_DATA, PHASE_TUNE_BWD_WEIGHT, PHASE_EVAL_FWD, PHASE_EVAL_BWD,
 PHASE_DEPLOY_FWD, PHASE_DEPLOY_BWD, PHASE_TUNE_BWD) = range(8)

EXPORTS = (
    "convbn_out_shape", "convbn_saved_bytes", "convbn_workspace_bytes", "convbn_tune_fwd",
    "convbn_tune_bwd_data", "convbn_tune_bwd_weight", "convbn_eval_fwd", "convbn_eval_bwd",
    "convbn_deploy_prepare", "convbn_deploy_fwd", "convbn_deploy_bwd", "convbn_check",
    "convbn_status_string", "convbn_last_kernel", "convbn_host_step_arena_bytes",
    "convbn_tune_step_host", "convbn_tune_step_host_begin", "convbn_tune_step_host_join", "convbn_profile_begin", "convbn_profile_end",
    "convbn_tune_bwd_weight_noalloc", "convbn_selftest_wait_timeout", "convbn_tune_bwd", "convbn_linear_desc", "convbn_relu", "convbn_add_relu", "convbn_relu_bwd", "convbn_add",
    "convbn_tune_bwd_begin", "convbn_tune_bwd_join",
    "convbn_tconv_out_shape", "convbn_tconv_workspace_bytes", "convbn_tconv_tune_fwd", "convbn_tconv_tune_bwd",
)


class ConvBNError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class Desc(ctypes.Structure):
    """Mirror of ``convbn_desc``."""
    _fields_ = [(k, ctypes.c_int) for k in (
        "n", "c_in", "h_in", "w_in", "c_out", "kh", "kw", "stride_h", "stride_w", "pad_h", "pad_w",
        "dil_h", "dil_w", "groups", "dtype", "layout")] + [("eps", ctypes.c_double)]

    @classmethod
    def make(cls, n, c_in, h_in, w_in, c_out, kh, kw, stride_h=1, stride_w=1, pad_h=0, pad_w=0,
             dil_h=1, dil_w=1, groups=1, dtype=BF16, layout=NHWC, eps=1e-5):
        return cls(n, c_in, h_in, w_in, c_out, kh, kw, stride_h, stride_w, pad_h, pad_w, dil_h,
                   dil_w, groups, dtype, layout, float(eps))


_lib = None


def lib():
    """Load the compiled library (raises OSError with the build hint if it is absent)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIBRARY):
            raise OSError("%s not found: run `python -m paper_2305_11624_b200.build` "
                          "(there is no CPU fallback)" % LIBRARY)
        L = ctypes.CDLL(LIBRARY)
        L.convbn_saved_bytes.restype = ctypes.c_size_t
        L.convbn_workspace_bytes.restype = ctypes.c_size_t
        L.convbn_host_step_arena_bytes.restype = ctypes.c_size_t
        L.convbn_status_string.restype = ctypes.c_char_p
        L.convbn_last_kernel.restype = ctypes.c_char_p
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def _ptr(t) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(None)
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _raise(status: int, where: str):
    if status != OK:
        raise ConvBNError(status, where)


def status_string(status: int) -> str:
    return lib().convbn_status_string(ctypes.c_int(status)).decode()


def convbn_last_kernel(phase: int) -> str:
    return lib().convbn_last_kernel(ctypes.c_int(phase)).decode()


def convbn_out_shape(desc: Desc):
    ho, wo = ctypes.c_int(0), ctypes.c_int(0)
    _raise(lib().convbn_out_shape(ctypes.byref(desc), ctypes.byref(ho), ctypes.byref(wo)),
           "convbn_out_shape")
    return ho.value, wo.value


def convbn_linear_desc(rows: int, in_features: int, out_features: int, dtype: int = BF16, eps: float = 1e-5) -> Desc:
    """Descriptor under which the convolution entry points compute a Linear-BN block on a [rows, in] matrix."""
    d = Desc()
    _raise(lib().convbn_linear_desc(ctypes.c_int(rows), ctypes.c_int(in_features), ctypes.c_int(out_features),
                                    ctypes.c_int(dtype), ctypes.c_double(eps), ctypes.byref(d)), "convbn_linear_desc")
    return d


def convbn_saved_bytes(desc: Desc, mode: int) -> int:
    return int(lib().convbn_saved_bytes(ctypes.byref(desc), ctypes.c_int(mode)))


def convbn_workspace_bytes(desc: Desc, phase: int) -> int:
    return int(lib().convbn_workspace_bytes(ctypes.byref(desc), ctypes.c_int(phase)))


def convbn_tune_fwd(desc, x, w, b, gamma, beta, run_mean, run_var, z, saved, workspace=None,
                    workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tune_fwd(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(b), _ptr(gamma),
                                 _ptr(beta), _ptr(run_mean), _ptr(run_var), _ptr(z), _ptr(saved),
                                 _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)),
           "convbn_tune_fwd")


def convbn_tune_bwd_data(desc, dz, w, saved, dx, workspace=None,
                         workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tune_bwd_data(ctypes.byref(desc), _ptr(dz), _ptr(w), _ptr(saved), _ptr(dx),
                                      _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)),
           "convbn_tune_bwd_data")


def convbn_tune_bwd_weight(desc, dz, x, w, b, run_mean, saved, dw, db, dgamma, dbeta,
                           workspace=None, workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tune_bwd_weight(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w), _ptr(b),
                                        _ptr(run_mean), _ptr(saved), _ptr(dw), _ptr(db),
                                        _ptr(dgamma), _ptr(dbeta), _ptr(workspace),
                                        ctypes.c_size_t(wb), _stream(stream)),
           "convbn_tune_bwd_weight")


def convbn_tune_bwd(desc, dz, x, w, b, run_mean, saved, dx, dw, db, dgamma, dbeta, workspace=None,
                    workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tune_bwd(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w), _ptr(b), _ptr(run_mean),
                                 _ptr(saved), _ptr(dx), _ptr(dw), _ptr(db), _ptr(dgamma), _ptr(dbeta),
                                 _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)),
           "convbn_tune_bwd")


def convbn_tune_bwd_begin(desc, dz, x, w, b, run_mean, saved, dx, dw, db, dgamma, dbeta, workspace=None,
                          workspace_bytes: Optional[int] = None, stream=None):
    """convbn_tune_bwd that returns with the parameter-gradient pass still running on the library's side lane."""
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tune_bwd_begin(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w), _ptr(b), _ptr(run_mean),
                                       _ptr(saved), _ptr(dx), _ptr(dw), _ptr(db), _ptr(dgamma), _ptr(dbeta),
                                       _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)), "convbn_tune_bwd_begin")


def convbn_tune_bwd_join(stream=None) -> None:
    """Make `stream` wait for every parameter-gradient pass begun by this thread on the current device."""
    _raise(lib().convbn_tune_bwd_join(_stream(stream)), "convbn_tune_bwd_join")


def convbn_tconv_out_shape(desc):
    h, w = ctypes.c_int(0), ctypes.c_int(0)
    _raise(lib().convbn_tconv_out_shape(ctypes.byref(desc), ctypes.byref(h), ctypes.byref(w)), "convbn_tconv_out_shape")
    return h.value, w.value


def convbn_tconv_workspace_bytes(desc) -> int:
    f = lib().convbn_tconv_workspace_bytes
    f.restype = ctypes.c_size_t
    return int(f(ctypes.byref(desc)))


def convbn_tconv_tune_fwd(desc, x, w, b, gamma, beta, run_mean, run_var, z, saved, workspace=None,
                          workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tconv_tune_fwd(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(b), _ptr(gamma), _ptr(beta),
                                       _ptr(run_mean), _ptr(run_var), _ptr(z), _ptr(saved), _ptr(workspace),
                                       ctypes.c_size_t(wb), _stream(stream)), "convbn_tconv_tune_fwd")


def convbn_tconv_tune_bwd(desc, dz, x, w, b, run_mean, saved, dx, dw, db, dgamma, dbeta, workspace=None,
                          workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_tconv_tune_bwd(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w), _ptr(b), _ptr(run_mean),
                                       _ptr(saved), _ptr(dx), _ptr(dw), _ptr(db), _ptr(dgamma), _ptr(dbeta),
                                       _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)), "convbn_tconv_tune_bwd")


def convbn_tune_bwd_weight_noalloc(desc, dz, x, w, b, run_mean, saved, dw, db, dgamma, dbeta,
                                   stream=None):
    """Same results as convbn_tune_bwd_weight for callers that must not allocate device memory:
    no workspace argument, the library's built-in 16 MiB scratch array is used instead.  Raises
    ConvBNError(ECAPACITY) when the layer needs more scratch than that.  Calls sharing a device
    must not overlap on it."""
    _raise(lib().convbn_tune_bwd_weight_noalloc(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w),
                                                _ptr(b), _ptr(run_mean), _ptr(saved), _ptr(dw),
                                                _ptr(db), _ptr(dgamma), _ptr(dbeta), _stream(stream)),
           "convbn_tune_bwd_weight_noalloc")


def convbn_eval_fwd(desc, x, w, b, gamma, beta, run_mean, run_var, z, y_saved, workspace=None,
                    workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_eval_fwd(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(b), _ptr(gamma),
                                 _ptr(beta), _ptr(run_mean), _ptr(run_var), _ptr(z), _ptr(y_saved),
                                 _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)),
           "convbn_eval_fwd")


def convbn_eval_bwd(desc, dz, x, y_saved, w, gamma, run_mean, run_var, dx, dw, db, dgamma, dbeta,
                    workspace=None, workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_eval_bwd(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(y_saved), _ptr(w),
                                 _ptr(gamma), _ptr(run_mean), _ptr(run_var), _ptr(dx), _ptr(dw),
                                 _ptr(db), _ptr(dgamma), _ptr(dbeta), _ptr(workspace),
                                 ctypes.c_size_t(wb), _stream(stream)),
           "convbn_eval_bwd")


def convbn_deploy_prepare(desc, w, b, gamma, beta, run_mean, run_var, w_fused, b_fused, stream=None):
    _raise(lib().convbn_deploy_prepare(ctypes.byref(desc), _ptr(w), _ptr(b), _ptr(gamma), _ptr(beta),
                                       _ptr(run_mean), _ptr(run_var), _ptr(w_fused), _ptr(b_fused),
                                       _stream(stream)),
           "convbn_deploy_prepare")


def convbn_deploy_fwd(desc, x, w_fused, b_fused, z, workspace=None,
                      workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_deploy_fwd(ctypes.byref(desc), _ptr(x), _ptr(w_fused), _ptr(b_fused), _ptr(z),
                                   _ptr(workspace), ctypes.c_size_t(wb), _stream(stream)),
           "convbn_deploy_fwd")


def convbn_deploy_bwd(desc, dz, x, w_fused, dx, dw_fused, db_fused, workspace=None,
                      workspace_bytes: Optional[int] = None, stream=None):
    wb = _nbytes(workspace) if workspace_bytes is None else workspace_bytes
    _raise(lib().convbn_deploy_bwd(ctypes.byref(desc), _ptr(dz), _ptr(x), _ptr(w_fused), _ptr(dx),
                                   _ptr(dw_fused), _ptr(db_fused), _ptr(workspace),
                                   ctypes.c_size_t(wb), _stream(stream)),
           "convbn_deploy_bwd")


def _dtype_of(t) -> int:
    import torch
    return {torch.bfloat16: BF16, torch.float16: F16}.get(t.dtype, F32)


def convbn_relu(a, out, stream=None):
    _raise(lib().convbn_relu(ctypes.c_int(_dtype_of(a)), _ptr(a), _ptr(out), ctypes.c_longlong(a.numel()), _stream(stream)),
           "convbn_relu")


def convbn_add_relu(a, b, out, stream=None):
    _raise(lib().convbn_add_relu(ctypes.c_int(_dtype_of(a)), _ptr(a), _ptr(b), _ptr(out), ctypes.c_longlong(a.numel()),
                                 _stream(stream)), "convbn_add_relu")


def convbn_relu_bwd(a, y, out, stream=None):
    _raise(lib().convbn_relu_bwd(ctypes.c_int(_dtype_of(a)), _ptr(a), _ptr(y), _ptr(out), ctypes.c_longlong(a.numel()),
                                 _stream(stream)), "convbn_relu_bwd")


def convbn_add(a, b, out, stream=None):
    _raise(lib().convbn_add(ctypes.c_int(_dtype_of(a)), _ptr(a), _ptr(b), _ptr(out), ctypes.c_longlong(a.numel()),
                            _stream(stream)), "convbn_add")


def convbn_check(stream=None) -> None:
    _raise(lib().convbn_check(_stream(stream)), "convbn_check")


def convbn_selftest_wait_timeout(stream=None) -> None:
    """Queue the failure-path self-test: the next convbn_check() raises ConvBNError(ETIMEOUT)."""
    _raise(lib().convbn_selftest_wait_timeout(_stream(stream)), "convbn_selftest_wait_timeout")


def convbn_host_step_arena_bytes(desc: Desc) -> int:
    return int(lib().convbn_host_step_arena_bytes(ctypes.byref(desc)))


def convbn_tune_step_host(desc, x, dz, w, b, gamma, beta, run_mean, run_var, z, dx, dw, db, dgamma,
                          dbeta, device_arena, arena_bytes: Optional[int] = None, stream=None):
    """All tensors but ``device_arena`` are HOST tensors (page-locked for asynchronous copies)."""
    ab = _nbytes(device_arena) if arena_bytes is None else arena_bytes
    _raise(lib().convbn_tune_step_host(ctypes.byref(desc), _ptr(x), _ptr(dz), _ptr(w), _ptr(b),
                                       _ptr(gamma), _ptr(beta), _ptr(run_mean), _ptr(run_var),
                                       _ptr(z), _ptr(dx), _ptr(dw), _ptr(db), _ptr(dgamma),
                                       _ptr(dbeta), _ptr(device_arena), ctypes.c_size_t(ab),
                                       _stream(stream)),
           "convbn_tune_step_host")


def convbn_tune_step_host_begin(desc, x, dz, w, b, gamma, beta, run_mean, run_var, z, dx, dw, db, dgamma,
                          dbeta, device_arena, arena_bytes: Optional[int] = None, stream=None):
    """All tensors but ``device_arena`` are HOST tensors (page-locked for asynchronous copies)."""
    ab = _nbytes(device_arena) if arena_bytes is None else arena_bytes
    _raise(lib().convbn_tune_step_host_begin(ctypes.byref(desc), _ptr(x), _ptr(dz), _ptr(w), _ptr(b),
                                       _ptr(gamma), _ptr(beta), _ptr(run_mean), _ptr(run_var),
                                       _ptr(z), _ptr(dx), _ptr(dw), _ptr(db), _ptr(dgamma),
                                       _ptr(dbeta), _ptr(device_arena), ctypes.c_size_t(ab),
                                       _stream(stream)),
           "convbn_tune_step_host_begin")


def convbn_tune_step_host_join(stream=None) -> None:
    """Make `stream` wait for the downloads of every convbn_tune_step_host_begin call of this thread on this device."""
    _raise(lib().convbn_tune_step_host_join(_stream(stream)), "convbn_tune_step_host_join")


def convbn_profile_begin() -> None:
    _raise(lib().convbn_profile_begin(), "convbn_profile_begin")


def convbn_profile_end() -> dict:
    """{kernel family: (launches, total milliseconds)} since convbn_profile_begin()."""
    buf = ctypes.create_string_buffer(1 << 16)
    _raise(lib().convbn_profile_end(buf, ctypes.c_size_t(len(buf))), "convbn_profile_end")
    out = {}
    for line in buf.value.decode().splitlines():
        name, count, ms = line.split()
        out[name] = (int(count), float(ms))
    return out
