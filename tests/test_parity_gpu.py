"""GPU parity: the CUDA library against the fp64 CPU oracle, element by element on the same
seeded inputs, through the C ABI.  Small shapes span several tiles, ragged tails and the
degenerate cases; the benchmark configurations run at full size."""
import numpy as np
import pytest

import parity
from oracle import oracle as O
from paper_2305_11624_b200 import inputs as I

pytestmark = pytest.mark.gpu

L = I.LayerSpec

SMALL = [
    # fp32 NCHW (direct kernels)
    L("f32_bias", 2, 16, 16, 16, 32, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True),
    L("f32_s2_g2", 3, 8, 13, 11, 12, 3, 3, stride=2, pad=1, groups=2, dtype="f32", layout="nchw", bias=True),
    L("f32_dil", 1, 5, 12, 9, 7, 3, 3, pad=2, dil=2, dtype="f32", layout="nchw"),
    L("f32_1x1", 2, 7, 5, 5, 3, 1, 1, dtype="f32", layout="nchw", bias=True),
    L("f32_one_pixel", 1, 4, 1, 1, 2, 3, 3, pad=1, dtype="f32", layout="nchw"),
    # bf16 NHWC: tensor-core eligible shapes (channels multiple of 64) with ragged pixel counts
    L("b_1x1_a", 3, 256, 9, 13, 64, 1, 1),
    L("b_1x1_b", 2, 64, 17, 15, 256, 1, 1),
    L("b_1x1_big", 1, 512, 20, 20, 192, 1, 1),
    L("b_3x3_a", 2, 64, 20, 24, 64, 3, 3, pad=1),
    L("b_3x3_b", 3, 128, 7, 7, 256, 3, 3, pad=1),
    L("b_3x3_s2", 2, 128, 21, 18, 128, 3, 3, stride=2, pad=1),
    L("b_3x3_nopad", 1, 64, 10, 11, 128, 3, 3),
    L("b_5x5", 1, 64, 12, 12, 64, 5, 5, pad=2),
    L("b_bias", 2, 64, 8, 8, 64, 3, 3, pad=1, bias=True),
    # bf16 NHWC: shapes that do not fit the tensor-core tiles
    L("b_odd_c", 2, 24, 9, 10, 40, 3, 3, pad=1),
    L("b_stem_like", 2, 3, 30, 30, 64, 7, 7, stride=2, pad=3),
    L("b_dil", 1, 64, 14, 14, 64, 3, 3, pad=2, dil=2),
    # depthwise / grouped
    L("b_dw", 2, 96, 14, 15, 96, 3, 3, pad=1, groups=96),
    L("b_dw_s2", 1, 32, 9, 9, 32, 3, 3, stride=2, pad=1, groups=32),
    L("b_grouped", 2, 256, 9, 9, 256, 3, 3, pad=1, groups=32),
    L("b_grouped_cout2x", 1, 16, 6, 6, 32, 3, 3, pad=1, groups=4),
    # strip kernel: column split (W > 256), BN = 128, ragged rows, 5x5, two channel chunks
    L("b_strip_wide", 1, 64, 7, 300, 64, 3, 3, pad=1),
    L("b_strip_bn128", 2, 128, 19, 33, 128, 3, 3, pad=1),
    L("b_strip_5x5", 1, 64, 21, 40, 64, 5, 5, pad=2),
    L("b_strip_1x3", 1, 64, 9, 30, 192, 1, 3, pad=0),
    # strided backward data: 1x1 stride 2 (empty residue classes), 5x5 stride 2, stride 3
    L("b_1x1_s2", 2, 64, 15, 14, 128, 1, 1, stride=2),
    L("b_5x5_s2", 1, 64, 17, 19, 64, 5, 5, stride=2, pad=2),
    L("b_3x3_s3", 1, 64, 20, 16, 64, 3, 3, stride=3, pad=1),
    # grouped block-diagonal with other group widths; depthwise 5x5
    L("b_grouped_cg4", 1, 64, 10, 12, 64, 3, 3, pad=1, groups=16),
    L("b_grouped_cg32_s2", 2, 128, 11, 9, 128, 3, 3, stride=2, pad=1, groups=4),
    L("b_dw_5x5", 1, 48, 11, 13, 48, 5, 5, pad=2, groups=48),
    # grouped, wide enough for the patch-reuse kernel (block-diagonal mode): two 64-channel blocks
    L("b_grouped_wide", 2, 128, 17, 22, 128, 3, 3, pad=1, groups=16),
    # 8 channels per group on warp-level MMAs: no padding, a 1x3 kernel (odd tap count), a bias
    L("b_grouped8_nopad", 1, 64, 12, 19, 64, 3, 3, pad=0, groups=8, bias=True),
    L("b_grouped8_1x3", 2, 128, 6, 33, 128, 1, 3, pad=1, groups=16),
    L("b_grouped8_2x2", 1, 64, 11, 14, 64, 2, 2, pad=0, groups=8),
    # depthwise 3x3 too narrow for the TMA row stream (W_out < 8): the register-streaming kernel
    L("b_dw_narrow", 2, 32, 9, 6, 32, 3, 3, pad=1, groups=32),
    L("b_dw_nopad", 3, 32, 13, 37, 32, 3, 3, pad=0, groups=32),
    L("b_dw_wide_c", 1, 256, 9, 21, 256, 3, 3, pad=1, groups=256),
    # narrow-input (stem) path: 4 and 8 input channels, two output-channel chunk groups, stride 1 and 3
    L("b_stem_c4", 1, 4, 19, 23, 128, 5, 5, pad=2),
    L("b_stem_c8_s3", 2, 8, 25, 22, 64, 3, 3, stride=3, pad=1),
    L("b_stem_3x3_s2", 1, 3, 41, 70, 64, 3, 3, stride=2, pad=1),
    # stride-2 backward data of narrow inputs as a sub-pixel convolution: one input channel with odd sizes
    # (unpaired stores), four channels with two output-channel chunks, no padding with input rows beyond
    # twice the output height
    L("b_sub_c1_odd", 2, 1, 33, 45, 64, 5, 5, stride=2, pad=2),
    L("b_sub_c4", 1, 4, 40, 64, 128, 7, 7, stride=2, pad=3),
    L("b_sub_nopad", 1, 3, 38, 52, 64, 4, 4, stride=2, pad=0),
    # stem forward with the windows formed by the operand addressing (W_in a multiple of 8, stride 2): three
    # channels with a ragged last chunk of rows, one and two channels, an output row wider than one M block,
    # 128 output channels, a 3x3 kernel without padding
    L("b_win_c3", 3, 3, 38, 48, 64, 7, 7, stride=2, pad=3),
    L("b_win_c1", 1, 1, 20, 32, 64, 5, 5, stride=2, pad=2, bias=True),
    L("b_win_c2_wide", 1, 2, 12, 272, 64, 3, 3, stride=2, pad=1),
    L("b_win_c4_128", 2, 4, 18, 40, 128, 3, 3, stride=2, pad=0),
    # ... an even kernel without padding whose last input row no output row reaches, four channels with 64 outputs
    L("b_win_tail", 2, 3, 21, 40, 64, 4, 4, stride=2, pad=0),
    L("b_win_c4_64", 3, 4, 26, 56, 64, 7, 7, stride=2, pad=3, bias=True),
    # the same regrouping for wide stride-2 layers: 128-column tiles; 64-column tiles with three
    # output-channel chunks, a 5x5 kernel and odd sizes
    L("b_sub_wide", 1, 128, 40, 58, 128, 3, 3, stride=2, pad=1),
    L("b_sub_wide_5x5", 1, 64, 37, 61, 192, 5, 5, stride=2, pad=2),
]

EXPECTED_PATH = {   # the specialised kernels must actually be the ones that ran
    "b_1x1_a": ("umma", "umma", "umma"), "b_3x3_a": ("umma-strip", "umma-strip", "umma"),
    "b_3x3_s2": ("umma", "umma-strided", "umma"), "b_dw": ("depthwise", "depthwise", "depthwise"),
    "b_grouped": ("grouped-mma", "grouped-mma", "grouped-mma"), "b_odd_c": ("direct", "direct", "direct"),
    "b_strip_wide": ("umma-strip", "umma-strip", "umma"), "b_strip_bn128": ("umma-strip", "umma-strip", "umma"),
    "b_1x1_s2": ("umma", "umma-strided", "umma"), "b_grouped_cg32_s2": ("grouped-umma", "direct", "grouped-umma"),
    "f32_bias": ("direct", "direct", "direct"),
    "b_stem_like": ("umma-stem", "stem-mma", "umma-stem"), "b_sub_c1_odd": ("umma-stem", "umma-subpixel", "umma-stem"),
    "b_sub_wide": ("umma", "umma-subpixel", "umma"), "b_sub_wide_5x5": ("umma", "umma-subpixel", "umma"),
    "b_sub_c4": ("umma-stem", "umma-subpixel", "umma-stem"), "b_sub_nopad": ("umma-stem", "umma-subpixel", "umma-stem"),
}


@pytest.mark.parametrize("spec", SMALL, ids=lambda s: s.name)
def test_tune_small(spec):
    t = parity.make_inputs(spec, 1234)
    ref = parity.oracle_tune(spec, t)
    got = parity.run_tune_gpu(spec, t)
    parity.compare(got, ref, parity.TOL[spec.dtype], parity.TUNE_OUTPUTS, spec.name, dtype=spec.dtype)
    if spec.name in EXPECTED_PATH:
        assert got["_kernels"] == EXPECTED_PATH[spec.name], got["_kernels"]


DEGENERATE = [sp for sp in SMALL if sp.name in ("f32_bias", "b_1x1_a", "b_3x3_a", "b_bias", "b_odd_c", "b_dw", "b_grouped",
                                               "b_win_c3", "b_sub_wide")] + \
    [L("h_3x3_64", 2, 64, 30, 30, 64, 3, 3, pad=1, dtype="f16", bias=True)]


@pytest.mark.parametrize("spec", DEGENERATE, ids=lambda s: s.name)
def test_degenerate_statistics_and_affine_parameters(spec):
    """The cases the rewrite itself can degenerate in (Sec. 3.3 definitions): gamma = 0 (the channel's omega' vanishes, its
    output is the constant b', its domega is zero while dgamma is not), negative gamma, a running variance of exactly
    zero (s = gamma / sqrt(eps), some 300 times larger than elsewhere) and a large one, a large running mean."""
    t = parity.make_inputs(spec, 4242)
    c = spec.c_out
    idx = np.arange(c)
    t["gamma"] = np.where(idx % 4 == 0, 0.0, np.where(idx % 4 == 1, -t["gamma"], t["gamma"])).astype(np.float32).astype(np.float64)
    t["var_hat"] = np.where(idx % 8 == 2, 0.0, np.where(idx % 8 == 3, 4096.0, t["var_hat"]))
    t["mu_hat"] = np.where(idx % 8 == 5, 37.5, t["mu_hat"])
    ref = parity.oracle_tune(spec, t)
    assert np.all(ref["w_f"][0] == 0.0) and np.all(ref["dw"][0] == 0.0) and np.abs(ref["dgamma"][0]) > 0
    got = parity.run_tune_gpu(spec, t)
    parity.compare(got, ref, parity.TOL[spec.dtype], parity.TUNE_OUTPUTS, spec.name, dtype=spec.dtype)
    assert np.all(got["dw"][0::4] == 0.0)                          # exactly
    # a channel with gamma = 0 outputs its b' everywhere, rounded once
    nchw_const = got["z"][:, 0]
    assert np.ptp(nchw_const) == 0.0 and abs(nchw_const.flat[0] - ref["b_f"][0]) <= 2.0 ** -8 * abs(ref["b_f"][0])


FULL = [(ci, li, sp) for ci, layers in I.CONFIGS.items() for li, sp in enumerate(layers)]


@pytest.mark.parametrize("ci,li,spec", FULL, ids=lambda v: v.name if isinstance(v, L) else None)
def test_tune_benchmark_configs_full_size(ci, li, spec):
    """All five configurations at full size, every element of every output tensor."""
    t = parity.make_inputs(spec, I.config_seed(ci, li))
    ref = parity.oracle_tune(spec, t)
    got = parity.run_tune_gpu(spec, t)
    errs = parity.compare(got, ref, parity.TOL[spec.dtype], parity.TUNE_OUTPUTS, spec.name, dtype=spec.dtype)
    print(spec.name, got["_kernels"], {k: "%.2e" % v for k, v in errs.items()})
    # the calls a benchmark step makes (backward in one call, parameter gradients joined afterwards), same bounds
    got = parity.run_tune_gpu(spec, t, deferred=True)
    parity.compare(got, ref, parity.TOL[spec.dtype], parity.TUNE_OUTPUTS, spec.name + " (begin / join)", dtype=spec.dtype)


def test_tune_is_deterministic_and_leaves_inputs_alone():
    from paper_2305_11624_b200.harness import Block
    import torch
    spec = L("det", 2, 64, 20, 24, 64, 3, 3, pad=1)
    t = parity.make_inputs(spec, 5)
    blk = Block(spec)
    blk.load(t)
    before = {k: getattr(blk, k).clone() for k in ("x", "w", "dz", "gamma", "beta", "mu_hat", "var_hat")}
    outs = []
    for _ in range(2):
        blk.tune_step()
        torch.cuda.synchronize()
        outs.append({k: getattr(blk, k).clone() for k in ("z", "dx", "dw", "dgamma", "dbeta")})
    for k in outs[0]:
        assert torch.equal(outs[0][k], outs[1][k]), k
    for k, v in before.items():
        assert torch.equal(getattr(blk, k), v), k


COMPARATOR_SPECS = [SMALL[0], SMALL[8], SMALL[10], SMALL[17], SMALL[19]] + \
    [sp for sp in SMALL if sp.name in ("b_stem_3x3_s2", "b_sub_c4", "b_sub_wide")] + \
    [I.find_layer(name)[2] for name in ("c1a", "c1b", "c1c", "c3c", "c4a")] + \
    [L("h_1x1_256_64", 2, 256, 28, 28, 64, 1, 1, dtype="f16"),                    # IEEE half in the three modes
     L("h_3x3_128_256", 2, 128, 20, 36, 256, 3, 3, pad=1, dtype="f16", bias=True),
     L("h_3x3_s2_128", 2, 128, 40, 42, 128, 3, 3, stride=2, pad=1, dtype="f16"),
     L("h_stem", 2, 3, 64, 80, 64, 7, 7, stride=2, pad=3, dtype="f16"),
     L("h_stem_w272", 2, 3, 8, 272, 64, 7, 7, stride=2, pad=3, dtype="f16", bias=True),
     L("h_20_24", 2, 20, 11, 13, 24, 3, 3, stride=2, pad=1, dtype="f16", bias=True),
     L("h_dw", 2, 96, 14, 15, 96, 3, 3, pad=1, groups=96, dtype="f16", bias=True),
     L("h_grouped8", 2, 256, 9, 9, 256, 3, 3, pad=1, groups=32, dtype="f16")]
# (the benchmark layers run at full size)


@pytest.mark.parametrize("spec", COMPARATOR_SPECS, ids=lambda s: s.name)
def test_eval_and_deploy_comparators(spec):
    """Eval and Deploy entry points against the oracle's Eval-row and Deploy-row equations (Table 2), at
    the same tolerance as the Tune path, and the paper's claim Z_eval = Z_deploy = Z_tune (Sec. 3.3) on
    the device outputs themselves."""
    from paper_2305_11624_b200.harness import Block
    from paper_2305_11624_b200 import convbn as C
    tol = parity.TOL[spec.dtype]
    t = parity.make_inputs(spec, 77)
    s = parity.oracle_shape(spec)
    p = dict(gamma=t["gamma"], beta=t["beta"], mu_hat=t["mu_hat"], var_hat=t["var_hat"])
    ev = O.eval_forward(s, t["x"], t["w"], t["b"], **p)
    ge = O.eval_backward(s, t["dz"], t["x"], ev["y"], t["w"], t["gamma"], t["mu_hat"], t["var_hat"],
                         with_bias=spec.bias)
    blk = Block(spec, modes=("tune", "eval", "deploy"))
    blk.load(t)
    blk.eval_fwd()
    z_eval = blk.fetch("z")
    errs = parity.compare({"y_saved": blk.fetch("y_saved"), "z": z_eval}, {"y_saved": ev["y"], "z": ev["z"]}, tol,
                          ("y_saved", "z"), spec.name + "/eval fwd", dtype=spec.dtype)
    blk.eval_bwd()
    got = {k: blk.fetch(k) for k in ("dx", "dw", "dgamma", "dbeta")}
    got["db"] = blk.fetch("db") if spec.bias else None
    errs.update(parity.compare(got, ge, tol, ("dx", "dw", "db", "dgamma", "dbeta"), spec.name + "/eval bwd",
                               dtype=spec.dtype, grads_from_stored=True))
    w_f, b_f = O.fold(s, t["w"], t["b"], **p)
    gd = O.deploy_backward(s, t["dz"], t["x"], w_f)
    blk.deploy_prepare(); blk.deploy_fwd()
    z_dep = blk.fetch("z")
    assert O.rel_l2(blk.fetch("w_fused"), w_f) <= tol
    assert O.rel_l2(blk.fetch("b_fused"), b_f) <= 1e-5
    parity.compare({"z": z_dep}, {"z": ev["z"]}, tol, ("z",), spec.name + "/deploy fwd", dtype=spec.dtype)
    blk.deploy_bwd()
    parity.compare({"dx": blk.fetch("dx"), "dw": blk.fetch("dw_fused"), "db": blk.fetch("db_fused")},
                   {"dx": gd["dx"], "dw": gd["dw_f"], "db": gd["db_f"]}, tol, ("dx", "dw", "db"),
                   spec.name + "/deploy bwd", dtype=spec.dtype)
    blk.tune_fwd()
    z_tune = blk.fetch("z")
    C.convbn_check()
    e_td, e_te = O.rel_l2(z_tune, z_dep), O.rel_l2(z_tune, z_eval)
    print(spec.name, {k: "%.2e" % v for k, v in errs.items()}, "tune~deploy %.2e tune~eval %.2e" % (e_td, e_te))
    assert e_td <= tol and e_te <= tol
    assert blk.saved_bytes("tune") < blk.saved_bytes("eval")
    assert blk.saved_bytes("tune") - blk.saved_bytes("deploy") == 3 * spec.c_out * 4
