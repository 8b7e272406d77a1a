"""IEEE-half storage (the paper's mixed-precision rows, Table 4): Tune-mode forward and backward of every kind of NHWC
layer against the fp64 oracle, inputs rounded to half on the host; half in the NCHW layout is refused.  (Eval and
Deploy mode in half: the half cases of test_parity_gpu.py and test_backbone_gpu.py.)"""
import numpy as np
import pytest
import torch

import parity
from paper_2305_11624_b200 import convbn as C
from paper_2305_11624_b200 import inputs as I
from paper_2305_11624_b200.harness import Block, make_desc

pytestmark = pytest.mark.gpu
L = I.LayerSpec

SHAPES = [
    L("h_1x1_256_64", 2, 256, 28, 28, 64, 1, 1, dtype="f16"),                       # fused single-read backward
    L("h_1x1_64_256", 2, 64, 28, 28, 256, 1, 1, dtype="f16", bias=True),
    L("h_1x1_512_128", 3, 512, 14, 14, 128, 1, 1, dtype="f16"),                      # two-call backward
    L("h_3x3_64", 2, 64, 30, 30, 64, 3, 3, pad=1, dtype="f16"),                      # strip kernel
    L("h_3x3_128_256", 2, 128, 20, 36, 256, 3, 3, pad=1, dtype="f16", bias=True),
    L("h_3x3_s2_128", 2, 128, 40, 42, 128, 3, 3, stride=2, pad=1, dtype="f16"),      # sub-pixel backward data
    L("h_3x3_256_7x7", 4, 256, 7, 7, 256, 3, 3, pad=1, dtype="f16"),                 # small images: im2col GEMM
    L("h_1x1_s2_256_512", 2, 256, 14, 14, 512, 1, 1, stride=2, dtype="f16"),         # residue-class backward data
    L("h_5x5_64_d2", 1, 64, 24, 24, 64, 5, 5, pad=4, dil=2, dtype="f16"),
    L("h_stem", 2, 3, 64, 80, 64, 7, 7, stride=2, pad=3, dtype="f16"),              # the three window kernels
]


# shapes the tensor-core kernels do not take: the direct kernels and the generic epilogue, instantiated for half
FALLBACK = [
    L("h_odd_48", 1, 48, 16, 16, 64, 3, 3, pad=1, dtype="f16"),
    L("h_20_24", 2, 20, 11, 13, 24, 3, 3, stride=2, pad=1, dtype="f16", bias=True),
    L("h_groups2", 1, 12, 9, 9, 10, 3, 3, pad=1, groups=2, dtype="f16"),
    # stems beyond the window kernels: packed forward and weight gradient; backward data by the sub-pixel route
    # (stride 2, at most 4 channels) or warp-level MMAs
    L("h_stem_w528", 1, 3, 8, 528, 64, 7, 7, stride=2, pad=3, dtype="f16"),
    L("h_stem_w272", 2, 3, 8, 272, 64, 7, 7, stride=2, pad=3, dtype="f16", bias=True),
    L("h_stem5_s1", 1, 3, 32, 32, 64, 5, 5, stride=1, pad=2, dtype="f16"),
    L("h_stem_c8_s2", 1, 8, 20, 24, 64, 3, 3, stride=2, pad=1, dtype="f16"),
    # depthwise: the row-streaming kernels (TMA ring; registers for narrow rows) and the general ones
    L("h_dw", 2, 96, 14, 15, 96, 3, 3, pad=1, groups=96, dtype="f16", bias=True),
    L("h_dw_narrow", 2, 32, 9, 6, 32, 3, 3, pad=1, groups=32, dtype="f16"),
    L("h_dw_s2", 1, 32, 9, 9, 32, 3, 3, stride=2, pad=1, groups=32, dtype="f16"),
    L("h_dw_5x5", 1, 48, 11, 13, 48, 5, 5, pad=2, groups=48, dtype="f16"),
    # grouped: warp-level MMAs (8 channels per group), block-diagonal tensor-core GEMMs (other widths)
    L("h_grouped8", 2, 256, 9, 9, 256, 3, 3, pad=1, groups=32, dtype="f16", bias=True),
    L("h_grouped_cg4", 1, 64, 10, 12, 64, 3, 3, pad=1, groups=16, dtype="f16"),
    L("h_grouped_cg32_s2", 2, 128, 11, 9, 128, 3, 3, stride=2, pad=1, groups=4, dtype="f16"),
    L("h_grouped_wide", 2, 128, 17, 22, 128, 3, 3, pad=1, groups=16, dtype="f16"),
]


@pytest.mark.parametrize("spec", SHAPES + FALLBACK, ids=lambda s: s.name)
def test_half_tune_against_the_oracle(spec):
    t = parity.make_inputs(spec, 4321)
    assert np.array_equal(t["x"], t["x"].astype(np.float16).astype(np.float32))      # the oracle reads what the GPU reads
    ref = parity.oracle_tune(spec, t)
    got = parity.run_tune_gpu(spec, t)
    errs = parity.compare(got, ref, parity.TOL["f16"], parity.TUNE_OUTPUTS, spec.name, dtype="f16")
    print(spec.name, got["_kernels"], {k: "%.1e" % v for k, v in errs.items()})
    if spec in SHAPES:
        assert all(k.startswith("umma") for k in got["_kernels"]), got["_kernels"]
    # the one-call backward gives the same numbers
    blk = Block(spec, modes=("tune",))
    blk.load(t)
    blk.tune_fwd(); blk.tune_bwd()
    C.convbn_check()
    two = {k: blk.fetch(k) for k in ("dx", "dw", "dgamma", "dbeta")}
    parity.compare(two, ref, parity.TOL["f16"], ("dx", "dw", "dgamma", "dbeta"), spec.name + " one call", dtype="f16")


def test_half_is_not_bf16():
    """The same bits read as the other 16-bit type give another tensor: a kernel that ignored the flag would fail."""
    spec = L("h_flag", 1, 64, 16, 16, 64, 3, 3, pad=1, dtype="f16")
    t = parity.make_inputs(spec, 7)
    got = parity.run_tune_gpu(spec, t)
    wrong = L("b_flag", 1, 64, 16, 16, 64, 3, 3, pad=1, dtype="bf16")
    blk = Block(wrong, modes=("tune",))
    hb = Block(spec, modes=("tune",)); hb.load(t)
    for name in ("x", "w", "dz"):
        getattr(blk, name).view(torch.int16).copy_(getattr(hb, name).view(torch.int16))      # half bits in bf16 buffers
    for name in ("gamma", "beta", "mu_hat", "var_hat"):
        getattr(blk, name).copy_(getattr(hb, name))
    blk.tune_fwd()
    C.convbn_check()
    z_bits_as_bf16 = blk.z.view(torch.int16).cpu().numpy()
    hb.tune_fwd()
    assert not np.array_equal(z_bits_as_bf16, hb.z.view(torch.int16).cpu().numpy())
    assert np.isfinite(got["z"]).all()


def test_half_is_an_nhwc_storage_type():
    """Half in the NCHW layout (the fp32 convention) is refused by every call, the size queries return 0."""
    d = make_desc(L("h_nchw", 1, 64, 16, 16, 64, 3, 3, pad=1, dtype="f16", layout="nchw"))
    assert C.convbn_workspace_bytes(d, C.PHASE_TUNE_FWD) == 0 and C.convbn_saved_bytes(d, C.MODE_EVAL) == 0
    for call in (C.convbn_tune_fwd, C.convbn_eval_fwd):
        with pytest.raises(C.ConvBNError) as e:
            call(d, 4096, 4096, None, 4096, 4096, 4096, 4096, 4096, 4096, 4096, 1 << 20, stream=0)
        assert e.value.status == C.EUNSUPPORTED


@pytest.mark.parametrize("name", ["c4a", "c4b"])
def test_half_depthwise_and_grouped_benchmark_layers_full_size(name):
    import dataclasses
    spec = dataclasses.replace(I.find_layer(name)[2], name=name + "_half", dtype="f16")
    t = parity.make_inputs(spec, 99)
    ref = parity.oracle_tune(spec, t)
    got = parity.run_tune_gpu(spec, t, deferred=True)
    errs = parity.compare(got, ref, parity.TOL["f16"], parity.TUNE_OUTPUTS, spec.name, dtype="f16")
    print(spec.name, got["_kernels"], {k: "%.1e" % v for k, v in errs.items()})


def test_half_glue_and_linear():
    a = torch.randn(4099, device="cuda:0").half(); b = torch.randn(4099, device="cuda:0").half()
    out = torch.empty_like(a)
    C.convbn_add_relu(a, b, out)
    C.convbn_check()
    ref = torch.relu(a.float() + b.float()).half()
    assert torch.equal(out, ref)
    d = C.convbn_linear_desc(1000, 128, 64, C.F16)
    assert (d.layout, d.dtype, d.c_in, d.c_out) == (C.NHWC, C.F16, 128, 64)
