"""convbn_tune_bwd: dX and the parameter gradients in one call (Table 2, Tune row) against the fp64 oracle.
The bottleneck's 1x1 layers run the kernel that reads dZ once; other layers run the two separate calls."""
import pytest

import parity
from paper_2305_11624_b200 import convbn as C
from paper_2305_11624_b200 import inputs as I
from paper_2305_11624_b200.harness import Block

pytestmark = pytest.mark.gpu

L = I.LayerSpec
SPECS = [
    (L("fb_256_64", 3, 256, 17, 15, 64, 1, 1), "umma-fused-bwd"),       # ragged last tile, several tiles per CTA
    (L("fb_64_256", 2, 64, 19, 21, 256, 1, 1), "umma-fused-bwd"),
    (L("fb_128_64", 2, 128, 16, 20, 64, 1, 1), "umma-fused-bwd"),
    (L("fb_64_128", 1, 64, 24, 30, 128, 1, 1), "umma-fused-bwd"),
    (L("fb_3x3", 2, 64, 12, 16, 64, 3, 3, pad=1), "two-calls"),
    (L("fb_f32", 2, 16, 8, 8, 32, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True), "two-calls"),
    (I.find_layer("c1a")[2], "umma-fused-bwd"),
    (I.find_layer("c1c")[2], "umma-fused-bwd"),
]


@pytest.mark.parametrize("spec,path", SPECS, ids=lambda v: v.name if isinstance(v, L) else None)
def test_tune_bwd_matches_the_oracle(spec, path):
    t = parity.make_inputs(spec, 99)
    ref = parity.oracle_tune(spec, t)
    blk = Block(spec)
    blk.load(t)
    blk.tune_fwd()
    for name in ("dx", "dw", "dgamma", "dbeta"):
        getattr(blk, name).fill_(float("nan"))           # the call must write every output itself
    blk.tune_bwd()
    C.convbn_check()
    assert C.convbn_last_kernel(C.PHASE_TUNE_BWD) == path
    names = ["dx", "dw", "dgamma", "dbeta"] + (["db"] if spec.bias else [])
    got = {k: blk.fetch(k) for k in names}
    got["db"] = got.get("db")
    errs = parity.compare(got, ref, parity.TOL[spec.dtype], ("dx", "dw", "db", "dgamma", "dbeta"), spec.name, dtype=spec.dtype)
    print(spec.name, {k: "%.2e" % v for k, v in errs.items()})


def test_tune_bwd_is_deterministic():
    import torch
    spec = SPECS[0][0]
    blk = Block(spec)
    blk.load(parity.make_inputs(spec, 5))
    blk.tune_fwd()
    outs = []
    for _ in range(2):
        blk.tune_bwd()
        torch.cuda.synchronize()
        outs.append({k: getattr(blk, k).clone() for k in ("dx", "dw", "dgamma", "dbeta")})
    for k in outs[0]:
        assert torch.equal(outs[0][k], outs[1][k]), k
