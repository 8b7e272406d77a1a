"""Shared helper of the GPU parity tests: run one layer through the CUDA library and through the
fp64 CPU oracle on the same seeded inputs and compare every output tensor by relative L2."""
import numpy as np

from oracle import oracle as O
from paper_2305_11624_b200 import inputs as I

# Tolerances: relative L2 per output tensor against the fp64 oracle.  bf16: inputs, omega' (backward
# data) and outputs are each rounded once to 8 mantissa bits (2^-9 = 2e-3 rms-ish each) -> 5e-3;
# fp32: sums of <= a few thousand products in fp32 -> 1e-5.
# f16 (IEEE half, 11 significant bits): omega' and the output are each rounded once at 2^-11 relative, which gives
# about 4e-4 in relative L2; the bound is set at 1e-3, five times tighter than the bf16 one.
TOL = {"bf16": 5e-3, "f32": 1e-5, "f16": 1e-3}


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


# Per-element bounds beside the norm (a relative L2 over millions of elements cannot see a few wrong
# pixels).  The scale of an element is max(|ref|, rms of ref over the element's CHANNEL): the per-channel
# factor s spreads the channels' magnitudes over a factor of four, and an error is proportional to its own
# channel's magnitude.  bf16 activations: the output rounding is at most 2^-8 |ref|; the rounded omega'
# and the fp32 accumulation add a random error with sigma of about 1.7e-3 of the channel rms per element,
# whose largest value over 10^7 elements stays below 5.5 sigma = 1e-2: the bound 2^-6 leaves a factor 1.5
# and still flags any element that is off by a sixty-fourth of its channel's scale.  fp32 tensors
# (config 0 activations, every parameter gradient): sums in fp32 of exact products, 1e-4 of scale.
# f16: roundings of 2^-11 instead of 2^-8, so sigma is about 2.8e-4 of the channel rms and 5.5 sigma = 1.5e-3; 2^-8
# leaves the factor 2.5 that a strided backward pass needs (three quarters of its dX are exact zeros, which halves
# the channel rms the errors of the other quarter are measured against).
ELEM_BOUND = {"bf16": 2.0 ** -6, "f32": 1e-4, "f16": 2.0 ** -8}
ACTIVATIONS = ("z", "dx", "y_saved")


def elem_excess(got, ref, bound, channel_axis=None):
    """max over elements of |got - ref| / (bound * max(|ref|, rms(ref over the channel))): <= 1 passes."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    if channel_axis is None or ref.ndim < 2:
        rms = np.sqrt(np.mean(ref * ref))
    else:
        axes = tuple(a for a in range(ref.ndim) if a != channel_axis)
        rms = np.sqrt(np.mean(ref * ref, axis=axes, keepdims=True))
    scale = np.maximum(np.abs(ref), rms)
    scale = np.where(scale == 0.0, 1.0, scale)
    return float(np.max(np.abs(got - ref) / (bound * scale)))


def compare(got: dict, ref: dict, tol: float, names, label="", dtype=None, grads_from_stored=False):
    """Relative L2 per tensor <= tol and, when `dtype` ("bf16" / "f32": the storage type of the
    activations) is given, the per-element bound ELEM_BOUND on every element.  grads_from_stored: the
    parameter gradients were formed from activations that went through the storage type on the way (Eval
    mode: Y and dY = s dZ are stored tensors), so they carry the storage type's rounding noise and get its
    bound; Tune and Deploy reduce fp32 accumulators of exact products and get the fp32 bound."""
    errs, worst = {}, {}
    for k in names:
        if ref.get(k) is None:
            assert got.get(k) is None
            continue
        errs[k] = O.rel_l2(got[k], ref[k])
        if dtype is not None:
            kind = dtype if (k in ACTIVATIONS or grads_from_stored) else "f32"
            # activations are [N, C, H, W], weights [C_out, ...] in logical order
            worst[k] = elem_excess(got[k], ref[k], ELEM_BOUND[kind], 1 if k in ACTIVATIONS else (0 if k == "dw" else None))
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "%s rel-L2 over %g: %r (all: %r)" % (label, tol, bad, errs)
    bad = {k: v for k, v in worst.items() if not (v <= 1.0)}
    assert not bad, "%s per-element bound exceeded (multiples of the bound): %r (all: %r)" % (label, bad, worst)
    return errs


def run_tune_gpu(spec, t, device="cuda:0", deferred=False):
    """Tune forward + backward through the library.  deferred=False: the three separate calls; True: the calls a
    benchmark step makes (convbn_tune_fwd, convbn_tune_bwd_begin, convbn_tune_bwd_join)."""
    from paper_2305_11624_b200.harness import Block
    from paper_2305_11624_b200 import convbn as C
    blk = Block(spec, device=device, modes=("tune",))
    blk.load(t)
    if deferred:
        blk.tune_fwd(); blk.tune_bwd_begin(); C.convbn_tune_bwd_join()
    else:
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
