"""Tensors beyond 2^31 elements (and 2^32 bytes): every index and byte offset has to be 64 bits wide.

A convolution does not mix images, so a batch made of R copies of a small batch has outputs that are R copies of the
small batch's outputs and parameter gradients that are R times the small batch's.  The fp64 oracle computes the small
batch in full; the library computes the big one; copies of the small outputs are compared with the oracle at the
first image, at the one that contains element 2^31, and at the last, and all copies are compared with the first."""
import numpy as np
import pytest
import torch

import parity
from oracle import oracle as O
from paper_2305_11624_b200 import convbn as C
from paper_2305_11624_b200 import inputs as I
from paper_2305_11624_b200.harness import Block

pytestmark = pytest.mark.gpu
L = I.LayerSpec

CASES = [
    # 1x1, 64 -> 128: Z and dZ hold 4.8e9 elements (9.7 GB each); the one-kernel backward pass
    (L("big_1x1", 1, 64, 256, 256, 128, 1, 1, bias=True), 576),
    # 3x3, 64 -> 64: 2.4e9 elements per tensor; strip kernel forward and backward data, split weight gradient
    (L("big_3x3", 2, 64, 128, 128, 64, 3, 3, pad=1), 1100),
]


@pytest.mark.parametrize("small,reps", CASES, ids=lambda v: v.name if isinstance(v, L) else str(v))
def test_batches_beyond_two_to_the_31_elements(small, reps):
    t = parity.make_inputs(small, 2024)
    ref = parity.oracle_tune(small, t)
    sb = Block(small, modes=("tune",))
    sb.load(t)
    big_spec = L(small.name + "_x%d" % reps, small.n * reps, small.c_in, small.h_in, small.w_in, small.c_out, small.kh,
                 small.kw, stride=small.stride, pad=small.pad, bias=small.bias)
    bb = Block(big_spec, modes=("tune",), allocate="params")
    for name in ("w", "gamma", "beta", "mu_hat", "var_hat") + (("b",) if small.bias else ()):
        getattr(bb, name).copy_(getattr(sb, name))
    bb.x, bb.dz = sb.x.repeat(reps), sb.dz.repeat(reps)
    assert max(bb.x.numel(), bb.dz.numel()) > 2 ** 31
    nan = lambda n: torch.full((n,), float("nan"), dtype=bb.tdtype, device=bb.device)
    bb.z, bb.dx = nan(bb.dz.numel()), nan(bb.x.numel())
    bb.saved = torch.empty(max(16, C.convbn_saved_bytes(bb.desc, C.MODE_TUNE)), dtype=torch.uint8, device=bb.device)
    bb.with_scratch(C.PHASE_TUNE_FWD, bb.tune_fwd)
    bb.with_scratch(C.PHASE_TUNE_BWD, bb.tune_bwd)
    C.convbn_check()
    tol = parity.TOL[small.dtype]
    for name, src in (("z", bb.z), ("dx", bb.dx)):
        per = src.numel() // reps
        across = (2 ** 31) // per                    # the copy that holds element 2^31
        assert 0 < across < reps - 1
        for i in (0, across, reps - 1):
            getattr(sb, name).copy_(src[i * per:(i + 1) * per])
            parity.compare({name: sb.fetch(name)}, ref, tol, (name,), "%s copy %d" % (big_spec.name, i), dtype=small.dtype)
        rows = src.view(reps, per).view(torch.int16)
        assert bool((rows == rows[0:1]).all()), name + ": copies differ"
    got = {k: bb.fetch(k) / reps for k in ("dw", "dgamma", "dbeta") + (("db",) if small.bias else ())}
    got.setdefault("db", None)
    errs = parity.compare(got, ref, tol, ("dw", "db", "dgamma", "dbeta"), big_spec.name)
    print(big_spec.name, {k: "%.1e" % v for k, v in errs.items()})


def test_glue_beyond_two_to_the_32_bytes():
    n = 2 ** 31 + 4099                                 # bf16: 4.3e9 bytes
    g = torch.Generator(device="cuda:0"); g.manual_seed(9)
    a = torch.randn(1 << 20, generator=g, device="cuda:0").to(torch.bfloat16).repeat(2049)[:n].contiguous()
    b = a.flip(0)
    out = torch.empty_like(a)
    C.convbn_add_relu(a, b, out)
    C.convbn_check()
    for lo in (0, 2 ** 31 - 4096, n - 8192):           # fp32 sum rounded once, as the kernel does
        want = torch.relu(a[lo:lo + 8192].float() + b[lo:lo + 8192].float()).to(torch.bfloat16)
        assert torch.equal(out[lo:lo + 8192], want), lo
    assert bool((out >= 0).all())
