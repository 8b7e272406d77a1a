"""Whole-backbone replay: a slice of three bottlenecks (one with a strided projection shortcut) chained through
the library - ConvBN blocks in Tune mode, ReLUs and skip connections - against the fp64 oracle chained the same
way, and the three modes against each other (Sec. 3.3 / 3.4: same function, different memory)."""
import numpy as np
import pytest
import torch

import parity
from oracle import oracle as O
from paper_2305_11624_b200 import inputs as I
from paper_2305_11624_b200.backbone import BackboneReplay, Bottleneck, resnet50_plan

pytestmark = pytest.mark.gpu

PLAN = [Bottleneck(64, 64, 256, 1, (12, 12)), Bottleneck(256, 64, 256, 1, (12, 12)), Bottleneck(256, 128, 512, 2, (12, 12))]


def _params(layer):
    b = layer.blk
    p = {k: b.fetch(k) for k in ("w", "gamma", "beta", "mu_hat", "var_hat")}
    p["shape"] = parity.oracle_shape(b.spec)
    return p


def _cb_fwd(p, x):
    return O.tune_forward(p["shape"], x, p["w"], None, gamma=p["gamma"], beta=p["beta"], mu_hat=p["mu_hat"], var_hat=p["var_hat"])


def _cb_bwd(p, dz, x, w_f):
    return O.tune_backward(p["shape"], dz, x, p["w"], w_f, None, p["gamma"], p["mu_hat"], p["var_hat"])


BODY = resnet50_plan(64)[1]        # all 16 bottlenecks of a ResNet-50 on 64 x 64 images: 16 x 16 down to 2 x 2 pixels


@pytest.mark.parametrize("mode,plan,dtype", [("tune", PLAN, "bf16"), ("eval", PLAN, "bf16"), ("deploy", PLAN, "bf16"),
                                             ("tune", BODY, "bf16"), ("tune", PLAN, "f16"), ("tune", BODY, "f16"),
                                             ("eval", PLAN, "f16"), ("deploy", PLAN, "f16")],
                         ids=["tune", "eval", "deploy", "tune_whole_body", "tune_half", "tune_whole_body_half",
                              "eval_half", "deploy_half"])
def test_three_bottlenecks_against_the_chained_oracle(mode, plan, dtype):
    """The three modes compute one function with one set of input gradients (Sec. 3.3), so one oracle chain - the
    Tune formulas - checks all of them; Deploy's parameter gradients belong to the folded parameters and are left
    to the per-layer tests.  The last case chains all 52 blocks of the network body (images down to 2 x 2 pixels)."""
    PLAN = plan
    ch_in, hw0, ch_out, hw1 = plan[0].c_in, plan[0].hw, plan[-1].c_out, (plan[-1].hw[0] // plan[-1].stride, plan[-1].hw[1] // plan[-1].stride)
    rp = BackboneReplay(2, PLAN, mode, seed=3, dtype=dtype)
    ins = rp.make_inputs(5)
    keep = {}
    rp.forward_backward(ins, keep)
    torch.cuda.synchronize()
    nchw = lambda t, c, hw: I.act_from_layout(t.float().cpu().numpy().astype(np.float64), "nhwc", (2, c, hw[0], hw[1]))
    x = nchw(ins["x"], ch_in, hw0)
    relu = lambda a: np.maximum(a, 0.0)
    tape = []
    for c1, c2, c3, ds in rp.blocks:
        P = [_params(l) if l is not None else None for l in (c1, c2, c3, ds)]
        f1 = _cb_fwd(P[0], x); a = relu(f1["z"])
        f2 = _cb_fwd(P[1], a); b = relu(f2["z"])
        f3 = _cb_fwd(P[2], b)
        fd = _cb_fwd(P[3], x) if ds is not None else None
        out = relu(f3["z"] + (fd["z"] if fd else x))
        tape.append((P, x, a, b, out, f1, f2, f3, fd))
        x = out
    g = nchw(ins["g"], ch_out, hw1)
    dw_first = dw_last = None
    # The sign of a pre-activation within rounding error of zero is decided by the arithmetic that produced it;
    # a flipped mask moves a whole gradient element, so both sides use the decisions the kernels took (their
    # stored ReLU outputs) while every value still comes from the oracle.
    masks = []
    for (ka, kb, kc), (P, xin, a, b, out, *_r) in zip(keep["relu_outputs"], tape):
        masks.append(tuple(nchw(t, ref.shape[1], ref.shape[2:]) > 0 for t, ref in ((ka, a), (kb, b), (kc, out))))
        for m, ref in zip(masks[-1], (a, b, out)):       # the decisions differ only where the oracle's value is tiny
            # (the per-element bound of one layer, doubled for the error the residual stream has gathered by the
            # third bottleneck and growing with the square root of the depth after that)
            lim = 2.0 ** -5 * max(1.0, np.sqrt(len(masks) / 3.0))
            assert np.abs(ref[m != (ref > 0)]).max(initial=0.0) <= lim * np.sqrt((ref * ref).mean())
    for (P, xin, a, b, out, f1, f2, f3, fd), (ma, mb, mo) in zip(reversed(tape), reversed(masks)):
        g = g * mo
        b3 = _cb_bwd(P[2], g, b, f3["w_f"]); gb = b3["dx"] * mb
        b2 = _cb_bwd(P[1], gb, a, f2["w_f"]); ga = b2["dx"] * ma
        b1 = _cb_bwd(P[0], ga, xin, f1["w_f"])
        gx = b1["dx"] + (_cb_bwd(P[3], g, xin, fd["w_f"])["dx"] if fd else g)
        if dw_last is None:
            dw_last = b3["dw"]
        dw_first = b1["dw"]
        g = gx
    depth = 3 * len(plan)           # convolutions on the longest path; rounding errors add in quadrature
    tol = parity.TOL[dtype] * np.sqrt(depth)
    got_out = nchw(keep["out"], ch_out, hw1)
    got_dx = nchw(keep["dx"], ch_in, hw0)
    errs = {"out": O.rel_l2(got_out, x), "dx": O.rel_l2(got_dx, g)}
    if mode != "deploy":
        errs["dw_first"] = O.rel_l2(rp.blocks[0][0].blk.fetch("dw"), dw_first)
        errs["dw_last"] = O.rel_l2(rp.blocks[-1][2].blk.fetch("dw"), dw_last)
    print(errs)
    assert all(v <= tol for v in errs.values()), errs


def test_modes_agree_and_eval_keeps_more():
    outs, peaks = {}, {}
    for mode in ("tune", "eval", "deploy"):
        rp = BackboneReplay(4, PLAN, mode, seed=3)
        ins = rp.make_inputs(5)
        keep = {}
        rp.forward_backward(ins, keep)
        torch.cuda.synchronize()
        outs[mode] = {k: keep[k].float().cpu().numpy().astype(np.float64) for k in ("out", "dx")}
        ms, peak, how = rp.measure(iters=2, warmup=1)
        peaks[mode] = peak
        assert ms > 0
    # Forward outputs agree closely.  The input gradients are compared with the oracle (above), not with each
    # other: between two modes the ReLU decisions of near-zero pre-activations differ in a fraction f of the
    # elements (about 0.3 % per layer in bf16), which moves a gradient by sqrt(2 f) per layer in relative L2.
    tol = parity.TOL["bf16"] * 3
    for mode in ("eval", "deploy"):
        assert O.rel_l2(outs["tune"]["out"], outs[mode]["out"]) <= tol, mode
        assert O.rel_l2(outs["tune"]["dx"], outs[mode]["dx"]) <= 0.3, mode
    # (at this size the per-call scratch outweighs the three vectors Tune keeps, so Tune and Deploy are not ordered)
    assert peaks["eval"] > 1.3 * max(peaks["tune"], peaks["deploy"]), peaks


def test_async_parameter_gradients_give_the_same_bits():
    outs = []
    for flag in (False, True):
        rp = BackboneReplay(2, PLAN, "tune", seed=3, async_param_grads=flag)
        ins = rp.make_inputs(5)
        keep = {}
        rp.forward_backward(ins, keep)
        torch.cuda.synchronize()
        outs.append((keep["out"], keep["dx"], [l.blk.dw.clone() for l in rp.layers], [l.blk.dgamma.clone() for l in rp.layers]))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    for a, b in zip(outs[0][2] + outs[0][3], outs[1][2] + outs[1][3]):
        assert torch.equal(a, b)


def test_resnet50_plan_has_53_blocks():
    stem, plan = resnet50_plan(224)
    rp_layers = 1 + sum(3 + (1 if (b.stride > 1 or b.c_in != b.c_out) else 0) for b in plan)
    assert rp_layers == 53 and plan[0].hw == (56, 56) and plan[-1].hw == (7, 7) and plan[-1].c_out == 2048


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("count", [0, 1, 7, 8, 4099, 148 * 1024 * 9 + 3])
def test_glue_operations_are_exact(dtype, count):
    """ReLU, add + ReLU, ReLU backward and add: one rounding of an exactly representable result, so bit equality
    with the same operation in numpy float64 rounded once to the storage type; ragged counts and in-place use."""
    from paper_2305_11624_b200 import convbn as C
    g = torch.Generator(device="cuda:0"); g.manual_seed(count + 1)
    pad = count + 8                    # keep a guard band behind the data: nothing past `count` may be written
    a = torch.randn(pad, generator=g, device="cuda:0").to(dtype)
    b = torch.randn(pad, generator=g, device="cuda:0").to(dtype)
    y = torch.randn(pad, generator=g, device="cuda:0").to(dtype)
    f = lambda t: t.float().cpu().numpy().astype(np.float64)
    back = lambda r: torch.from_numpy(r).to(dtype).float().numpy()     # round to nearest even, once
    fa, fb, fy = f(a), f(b), f(y)
    guard = -7.0
    for name, call, ref in (("relu", lambda o: C.convbn_relu(a, o), np.maximum(fa, 0)),
                            ("add_relu", lambda o: C.convbn_add_relu(a, b, o), np.maximum(fa + fb, 0)),
                            ("relu_bwd", lambda o: C.convbn_relu_bwd(a, y, o), fa * (fy > 0)),
                            ("add", lambda o: C.convbn_add(a, b, o), fa + fb)):
        out = torch.full((pad,), guard, dtype=dtype, device="cuda:0")
        view = out[:count]
        if count == 0:
            view = out[:0]
        # the binding takes the count from the first operand
        args_a, args_b, args_y = a[:count], b[:count], y[:count]
        {"relu": lambda: C.convbn_relu(args_a, view), "add_relu": lambda: C.convbn_add_relu(args_a, args_b, view),
         "relu_bwd": lambda: C.convbn_relu_bwd(args_a, args_y, view), "add": lambda: C.convbn_add(args_a, args_b, view)}[name]()
        C.convbn_check()
        got = out.float().cpu().numpy()
        assert np.array_equal(got[:count], back(ref[:count]) + 0.0), name       # (+0.0: -0 and +0 compare equal anyway)
        assert np.all(got[count:] == guard), name
    if count:
        inplace = a[:count].clone()
        C.convbn_add_relu(inplace, b[:count], inplace)
        C.convbn_check()
        assert np.array_equal(inplace.float().cpu().numpy(), back(np.maximum(fa + fb, 0)[:count]))
