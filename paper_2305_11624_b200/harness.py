"""Device-buffer bookkeeping for one ConvBN layer: allocation with torch, upload of synthetic
tensors in the layer's layout, calls through the binding, download in logical order.

Holds no arithmetic of the method: every step of a pass runs in ``libconvbn.so``.
"""
from typing import Dict, Optional

import numpy as np
import torch

from . import convbn as C
from . import inputs as I


def make_desc(spec: I.LayerSpec) -> C.Desc:
    return C.Desc.make(dtype={"bf16": C.BF16, "f16": C.F16}.get(spec.dtype, C.F32),
                       layout=C.NHWC if spec.layout == "nhwc" else C.NCHW, eps=spec.eps,
                       **spec.dims())


class Block:
    """Buffers of one layer on one device plus the calls of each mode."""

    def __init__(self, spec: I.LayerSpec, device="cuda:0", modes=("tune",), allocate="all"):
        """allocate="params" makes only the parameters and their gradients: activations, saved state and
        scratch are then assigned by the caller (memory measurements that allocate them per call)."""
        self.spec = spec
        self.desc = make_desc(spec)
        self.device = torch.device(device)
        self.h_out, self.w_out = C.convbn_out_shape(self.desc)
        self.tdtype = {"bf16": torch.bfloat16, "f16": torch.float16}.get(spec.dtype, torch.float32)
        cg = spec.c_in // spec.groups
        self.x_shape = (spec.n, spec.c_in, spec.h_in, spec.w_in)
        self.w_shape = (spec.c_out, cg, spec.kh, spec.kw)
        self.z_shape = (spec.n, spec.c_out, self.h_out, self.w_out)
        e = lambda shape, dt=self.tdtype: torch.empty(int(np.prod(shape)), dtype=dt, device=self.device)
        f = lambda: torch.empty(spec.c_out, dtype=torch.float32, device=self.device)
        self.w = e(self.w_shape)
        self.b = f() if spec.bias else None
        self.gamma, self.beta, self.mu_hat, self.var_hat = f(), f(), f(), f()
        self.dw = e(self.w_shape, torch.float32)
        self.db = f() if spec.bias else None
        self.dgamma, self.dbeta = f(), f()
        self.x = self.dz = self.z = self.dx = self.saved = self.y_saved = self.workspace = None
        if allocate == "params":
            return
        self.x, self.dz = e(self.x_shape), e(self.z_shape)
        self.z, self.dx = e(self.z_shape), e(self.x_shape)
        phases = []
        if "tune" in modes:
            phases += [C.PHASE_TUNE_FWD, C.PHASE_TUNE_BWD_DATA, C.PHASE_TUNE_BWD_WEIGHT, C.PHASE_TUNE_BWD]
            self.saved = torch.empty(max(16, C.convbn_saved_bytes(self.desc, C.MODE_TUNE)),
                                     dtype=torch.uint8, device=self.device)
        if "eval" in modes:
            phases += [C.PHASE_EVAL_FWD, C.PHASE_EVAL_BWD]
            self.y_saved = torch.empty(C.convbn_saved_bytes(self.desc, C.MODE_EVAL),
                                       dtype=torch.uint8, device=self.device)
        if "deploy" in modes:
            phases += [C.PHASE_DEPLOY_FWD, C.PHASE_DEPLOY_BWD]
            self.w_fused = e(self.w_shape)
            self.b_fused = f()
            self.dw_fused = e(self.w_shape, torch.float32)
            self.db_fused = f()
        ws = max([C.convbn_workspace_bytes(self.desc, p) for p in phases] + [256])
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.device)

    # ---- data movement ---------------------------------------------------------------------
    def _up(self, dst: torch.Tensor, a: np.ndarray):
        dst.copy_(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).reshape(-1).to(dst.dtype))

    def load(self, t: Dict[str, Optional[np.ndarray]]):
        """Upload logical-NCHW fp32 arrays (values already representable in the storage type)."""
        lay = self.spec.layout
        self._up(self.x, I.act_to_layout(t["x"], lay))
        self._up(self.dz, I.act_to_layout(t["dz"], lay))
        self._up(self.w, I.weight_to_layout(t["w"], lay))
        for name in ("gamma", "beta", "mu_hat", "var_hat"):
            self._up(getattr(self, name), t[name])
        if self.b is not None:
            self._up(self.b, t["b"])

    def randomize(self, seed: int):
        """Fill the inputs on the device with the recipe's distributions (for timing runs)."""
        g = self.randomize_params(seed)
        rn = lambda t, std: t.copy_((torch.randn(t.numel(), generator=g, device=self.device) * std).to(t.dtype))
        rn(self.x, 1.0); rn(self.dz, 1.0)

    def randomize_params(self, seed: int):
        """Fill the parameters only; returns the generator for further draws."""
        g = torch.Generator(device=self.device)
        g.manual_seed(seed)
        sp = self.spec
        fan_in = (sp.c_in // sp.groups) * sp.kh * sp.kw
        rn = lambda t, std: t.copy_((torch.randn(t.numel(), generator=g, device=self.device) * std).to(t.dtype))
        ru = lambda t, lo, hi: t.copy_(torch.rand(t.numel(), generator=g, device=self.device) * (hi - lo) + lo)
        rn(self.w, float(np.sqrt(2.0 / fan_in)))
        rn(self.mu_hat, 0.1); rn(self.beta, 0.1); ru(self.var_hat, 0.5, 2.0); ru(self.gamma, 0.5, 1.5)
        if self.b is not None:
            rn(self.b, 0.01)
        return g

    def with_scratch(self, phase: int, call):
        """Run one entry point with a workspace allocated for this call alone and released after it."""
        self.workspace = torch.empty(max(256, C.convbn_workspace_bytes(self.desc, phase)), dtype=torch.uint8,
                                     device=self.device)
        try:
            call()
        finally:
            self.workspace = None

    def fetch(self, name: str) -> np.ndarray:
        """Download a buffer as float64 in logical order."""
        t = getattr(self, name)
        a = t.detach().to(torch.float32).cpu().numpy().astype(np.float64)
        lay = self.spec.layout
        if name in ("x", "dx"):
            return I.act_from_layout(a, lay, self.x_shape)
        if name in ("z", "dz"):
            return I.act_from_layout(a, lay, self.z_shape)
        if name in ("w", "dw", "w_fused", "dw_fused"):
            return I.weight_from_layout(a, lay, self.w_shape)
        if name == "y_saved":
            a = t.view(self.tdtype).to(torch.float32).cpu().numpy().astype(np.float64)
            return I.act_from_layout(a, lay, self.z_shape)
        return a

    # ---- Tune mode -------------------------------------------------------------------------
    def tune_fwd(self, stream=None):
        C.convbn_tune_fwd(self.desc, self.x, self.w, self.b, self.gamma, self.beta, self.mu_hat,
                          self.var_hat, self.z, self.saved, self.workspace, stream=stream)

    def tune_bwd_data(self, stream=None):
        C.convbn_tune_bwd_data(self.desc, self.dz, self.w, self.saved, self.dx, self.workspace,
                               stream=stream)

    def tune_bwd_weight(self, stream=None):
        C.convbn_tune_bwd_weight(self.desc, self.dz, self.x, self.w, self.b, self.mu_hat, self.saved,
                                 self.dw, self.db, self.dgamma, self.dbeta, self.workspace,
                                 stream=stream)

    def tune_bwd(self, stream=None):
        C.convbn_tune_bwd(self.desc, self.dz, self.x, self.w, self.b, self.mu_hat, self.saved, self.dx, self.dw,
                          self.db, self.dgamma, self.dbeta, self.workspace, stream=stream)

    def tune_bwd_begin(self, stream=None):
        """Backward with the parameter-gradient pass left running on the library's side lane; dw, db, dgamma, dbeta and
        the workspace belong to it until C.convbn_tune_bwd_join(stream)."""
        C.convbn_tune_bwd_begin(self.desc, self.dz, self.x, self.w, self.b, self.mu_hat, self.saved, self.dx, self.dw,
                                self.db, self.dgamma, self.dbeta, self.workspace, stream=stream)

    def tune_step(self, stream=None, defer_join=False):
        self.tune_fwd(stream)
        if defer_join:
            self.tune_bwd_begin(stream)
        else:
            self.tune_bwd(stream)

    # ---- Eval mode -------------------------------------------------------------------------
    def eval_fwd(self, stream=None):
        C.convbn_eval_fwd(self.desc, self.x, self.w, self.b, self.gamma, self.beta, self.mu_hat,
                          self.var_hat, self.z, self.y_saved, self.workspace, stream=stream)

    def eval_bwd(self, stream=None):
        C.convbn_eval_bwd(self.desc, self.dz, self.x, self.y_saved, self.w, self.gamma, self.mu_hat,
                          self.var_hat, self.dx, self.dw, self.db, self.dgamma, self.dbeta,
                          self.workspace, stream=stream)

    # ---- Deploy mode -----------------------------------------------------------------------
    def deploy_prepare(self, stream=None):
        C.convbn_deploy_prepare(self.desc, self.w, self.b, self.gamma, self.beta, self.mu_hat,
                                self.var_hat, self.w_fused, self.b_fused, stream=stream)

    def deploy_fwd(self, stream=None):
        C.convbn_deploy_fwd(self.desc, self.x, self.w_fused, self.b_fused, self.z, self.workspace,
                            stream=stream)

    def deploy_bwd(self, stream=None):
        C.convbn_deploy_bwd(self.desc, self.dz, self.x, self.w_fused, self.dx, self.dw_fused,
                            self.db_fused, self.workspace, stream=stream)

    # ---- accounting ------------------------------------------------------------------------
    def flops_per_phase(self) -> float:
        sp = self.spec
        return 2.0 * sp.n * self.h_out * self.w_out * sp.c_out * (sp.c_in // sp.groups) * sp.kh * sp.kw

    def saved_bytes(self, mode: str) -> int:
        """Bytes kept from forward to backward beside nothing else: X plus the mode's extra."""
        es = 2 if self.spec.dtype in ("bf16", "f16") else 4
        xb = int(np.prod(self.x_shape)) * es
        m = {"tune": C.MODE_TUNE, "eval": C.MODE_EVAL, "deploy": C.MODE_DEPLOY}[mode]
        return xb + C.convbn_saved_bytes(self.desc, m)
