"""Shared helper of the GPU parity tests: run one layer through the CUDA library and through the
fp64 CPU oracle on the same seeded inputs and compare every output tensor by relative L2."""
import numpy as np

from oracle import oracle as O
from paper_2305_11624_b200 import inputs as I

# Tolerances: relative L2 per output tensor against the fp64 oracle.  bf16: inputs, omega' (backward
# data) and outputs are each rounded once to 8 mantissa bits (2^-9 = 2e-3 rms-ish each) -> 5e-3;
# fp32: sums of <= a few thousand products in fp32 -> 1e-5.
TOL = {"bf16": 5e-3, "f32": 1e-5}


def oracle_shape(spec: I.LayerSpec) -> O.Shape:
    return O.Shape(eps=spec.eps, **spec.dims())


def oracle_tune(spec, t):
    s = oracle_shape(spec)
    p = dict(gamma=t["gamma"], beta=t["beta"], mu_hat=t["mu_hat"], var_hat=t["var_hat"])
    fw = O.tune_forward(s, t["x"], t["w"], t["b"], **p)
    bw = O.tune_backward(s, t["dz"], t["x"], t["w"], fw["w_f"], t["b"], t["gamma"], t["mu_hat"], t["var_hat"])
    out = {"z": fw["z"], "w_f": fw["w_f"], "b_f": fw["b_f"]}
    out.update(bw)
    return out


def make_inputs(spec, seed):
    s = oracle_shape(spec)
    return I.make_block(spec, seed, O.out_hw(s))


def compare(got: dict, ref: dict, tol: float, names, label=""):
    errs = {}
    for k in names:
        if ref.get(k) is None:
            assert got.get(k) is None
            continue
        errs[k] = O.rel_l2(got[k], ref[k])
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "%s rel-L2 over %g: %r (all: %r)" % (label, tol, bad, errs)
    return errs


def run_tune_gpu(spec, t, device="cuda:0"):
    from paper_2305_11624_b200.harness import Block
    from paper_2305_11624_b200 import convbn as C
    blk = Block(spec, device=device, modes=("tune",))
    blk.load(t)
    blk.tune_fwd(); blk.tune_bwd_data(); blk.tune_bwd_weight()
    C.convbn_check()
    names = ["z", "dx", "dw", "dgamma", "dbeta"] + (["db"] if spec.bias else [])
    out = {k: blk.fetch(k) for k in names}
    if not spec.bias:
        out["db"] = None
    out["_kernels"] = tuple(C.convbn_last_kernel(p) for p in
                            (C.PHASE_TUNE_FWD, C.PHASE_TUNE_BWD_DATA, C.PHASE_TUNE_BWD_WEIGHT))
    return out


TUNE_OUTPUTS = ("z", "dx", "dw", "db", "dgamma", "dbeta")
