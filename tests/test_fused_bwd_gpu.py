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


def test_begin_join_gives_the_bits_of_the_synchronous_call():
    """convbn_tune_bwd_begin leaves the parameter-gradient passes of several layers on the side lane; after one
    convbn_tune_bwd_join every output equals the synchronous call's bit for bit (the kernels and their order of
    additions are the same), inside and outside a captured graph."""
    import torch
    specs = [s for s, _ in SPECS[:6]]
    blks = []
    for i, spec in enumerate(specs):
        b = Block(spec)
        b.load(parity.make_inputs(spec, 40 + i))
        b.tune_fwd()
        b.tune_bwd()
        blks.append(b)
    torch.cuda.synchronize()
    names = ("dx", "dw", "dgamma", "dbeta")
    want = [{k: getattr(b, k).clone() for k in names} for b in blks]

    def poison():
        for b in blks:
            for k in names:
                getattr(b, k).fill_(float("nan"))

    poison()
    for b in blks:
        b.tune_bwd_begin()
    C.convbn_tune_bwd_join()
    torch.cuda.synchronize()
    C.convbn_check()
    for b, w in zip(blks, want):
        for k in names:
            assert torch.equal(getattr(b, k), w[k]), (b.spec.name, k)
    C.convbn_tune_bwd_join()                               # nothing pending: a no-op

    poison()
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        for b in blks:
            b.tune_bwd_begin()
        C.convbn_tune_bwd_join()
    poison()
    gr.replay()
    torch.cuda.synchronize()
    C.convbn_check()
    for b, w in zip(blks, want):
        for k in names:
            assert torch.equal(getattr(b, k), w[k]), (b.spec.name, k, "graph")
