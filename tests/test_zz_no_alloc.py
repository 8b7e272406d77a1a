"""convbn_tune_bwd_weight_noalloc: the parameter-gradient call for users who may not allocate
device memory (allocator callbacks, plug-ins without their own memory, latency-critical loops).
It must return what convbn_tune_bwd_weight returns while using only the scratch array built into
the library, on repeated calls, and must refuse layers whose scratch need exceeds that array.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test."""
import numpy as np
import pytest
import torch

import parity
from paper_2305_11624_b200 import convbn as C
from paper_2305_11624_b200 import inputs as I
from paper_2305_11624_b200.harness import Block

pytestmark = pytest.mark.gpu

SPECS = [
    I.LayerSpec("na_f32", 2, 16, 16, 16, 32, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True),
    I.LayerSpec("na_bf16", 2, 64, 20, 24, 128, 3, 3, pad=1),
]


@pytest.mark.parametrize("spec", SPECS, ids=lambda s: s.name)
def test_noalloc_matches_workspace_variant_on_two_calls(spec):
    """Both entry points run the same kernels in the same fixed order, so the honest check is bit
    equality with the workspace call (anything stale in the shared scratch would break it), on two
    calls in a row, plus one comparison with the CPU oracle."""
    t = parity.make_inputs(spec, 31)
    blk = Block(spec)
    blk.load(t)
    blk.tune_fwd()
    blk.tune_bwd_weight()
    C.convbn_check()
    names = ["dw", "dgamma", "dbeta"] + (["db"] if spec.bias else [])
    want = {k: blk.fetch(k) for k in names}
    ref = parity.oracle_tune(spec, t)
    parity.compare(dict(want, db=want.get("db")), ref, parity.TOL[spec.dtype], ("dw", "db", "dgamma", "dbeta"),
                   spec.name + "/workspace call", dtype=spec.dtype)

    def call():
        for k in names:
            getattr(blk, k).fill_(float("nan"))      # the call must rewrite every output itself
        C.convbn_tune_bwd_weight_noalloc(blk.desc, blk.dz, blk.x, blk.w, blk.b, blk.mu_hat, blk.saved,
                                         blk.dw, blk.db, blk.dgamma, blk.dbeta)
        C.convbn_check()

    call()                                               # first call on this device: looks up the array's address
    torch.cuda.synchronize()
    # The library carries its own CUDA runtime, so torch's allocator statistics cannot see an allocation
    # made inside it; the driver's count of free device memory can.
    free_before = torch.cuda.mem_get_info()[0]
    for i in range(2):
        call()
        for k in names:
            got = blk.fetch(k)
            assert np.array_equal(got, want[k]), (k, i, float(np.max(np.abs(got - want[k]))))
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was allocated during the calls"


def test_noalloc_refuses_layers_beyond_its_scratch():
    big = C.Desc.make(8, 1024, 7, 7, 1024, 3, 3, pad_h=1, pad_w=1)
    assert C.convbn_workspace_bytes(big, C.PHASE_TUNE_BWD_WEIGHT) > 16 << 20
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tune_bwd_weight_noalloc(big, 4096, 4096, 4096, None, 4096, 4096, 4096, None, 4096, 4096,
                                         stream=0)
    assert e.value.status == C.ECAPACITY
    assert "16 MiB" in C.status_string(C.ECAPACITY)
