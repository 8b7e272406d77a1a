"""convbn_tune_step_host (host buffers in, host buffers out) against the fp64 oracle."""
import numpy as np
import pytest

from paper_2305_11624_b200 import inputs as I

import parity

pytestmark = pytest.mark.gpu

SPECS = [
    I.LayerSpec("h_3x3", 2, 64, 18, 20, 128, 3, 3, pad=1),
    I.LayerSpec("h_bias_f32", 2, 8, 9, 7, 12, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True),
    I.LayerSpec("h_dw", 1, 32, 13, 17, 32, 3, 3, pad=1, groups=32),
    I.LayerSpec("h_half_1x1", 2, 256, 20, 20, 64, 1, 1, dtype="f16", bias=True),
]


@pytest.mark.parametrize("spec", SPECS, ids=lambda s: s.name)
def test_host_step(spec):
    import torch
    from paper_2305_11624_b200 import convbn as C
    from paper_2305_11624_b200.harness import Block

    t = parity.make_inputs(spec, 77)
    ref = parity.oracle_tune(spec, t)
    blk = Block(spec, device="cuda:0", modes=("tune",))
    blk.load(t)                                        # device copies are only the templates of the host ones
    pin = lambda a: None if a is None else a.detach().cpu().pin_memory()
    out = lambda a: None if a is None else torch.zeros(a.shape, dtype=a.dtype).pin_memory()
    ins = [pin(a) for a in (blk.x, blk.dz, blk.w, blk.b, blk.gamma, blk.beta, blk.mu_hat, blk.var_hat)]
    outs = [out(a) for a in (blk.z, blk.dx, blk.dw, blk.db, blk.dgamma, blk.dbeta)]
    arena = torch.empty(C.convbn_host_step_arena_bytes(blk.desc), dtype=torch.uint8, device="cuda:0")
    for _ in range(2):                                 # twice: the second call reuses the arena and the copy lane
        C.convbn_tune_step_host(blk.desc, *ins, *outs, arena)
        torch.cuda.synchronize()
        C.convbn_check()
    # put the host results where Block.fetch reads them, to reuse its layout conversions
    for name, h in zip(("z", "dx", "dw", "db", "dgamma", "dbeta"), outs):
        if h is not None:
            getattr(blk, name).copy_(h)
    names = ["z", "dx", "dw", "dgamma", "dbeta"] + (["db"] if spec.bias else [])
    got = {k: blk.fetch(k) for k in names}
    if not spec.bias:
        got["db"] = None
    parity.compare(got, ref, parity.TOL[spec.dtype], parity.TUNE_OUTPUTS, spec.name, dtype=spec.dtype)


def test_pipelined_host_steps_give_the_bits_of_the_joined_call():
    """convbn_tune_step_host_begin on several layers (own arenas, then twice on ONE arena) and one join: every host
    output equals the joined call's, bit for bit."""
    import torch
    from paper_2305_11624_b200 import convbn as C
    from paper_2305_11624_b200 import inputs as I
    from paper_2305_11624_b200.harness import Block

    L = I.LayerSpec
    specs = [L("hp_1x1", 2, 256, 20, 20, 64, 1, 1), L("hp_3x3", 2, 64, 24, 24, 64, 3, 3, pad=1),
             L("hp_f32", 2, 16, 8, 8, 32, 3, 3, pad=1, dtype="f32", layout="nchw", bias=True)]
    layers = []
    for i, spec in enumerate(specs):
        blk = Block(spec, device="cuda:0", modes=("tune",))
        blk.load(parity.make_inputs(spec, 80 + i))
        pin = lambda a: None if a is None else a.detach().cpu().pin_memory()
        out = lambda a: None if a is None else torch.zeros(a.shape, dtype=a.dtype).pin_memory()
        ins = [pin(a) for a in (blk.x, blk.dz, blk.w, blk.b, blk.gamma, blk.beta, blk.mu_hat, blk.var_hat)]
        outs = [out(a) for a in (blk.z, blk.dx, blk.dw, blk.db, blk.dgamma, blk.dbeta)]
        arena = torch.empty(C.convbn_host_step_arena_bytes(blk.desc), dtype=torch.uint8, device="cuda:0")
        C.convbn_tune_step_host(blk.desc, *ins, *outs, arena)
        torch.cuda.synchronize()
        want = [None if o is None else o.clone() for o in outs]
        layers.append((blk, ins, outs, arena, want))
    for _, _, outs, _, _ in layers:
        for o in outs:
            if o is not None:
                o.fill_(float("nan"))
    for blk, ins, outs, arena, _ in layers:
        C.convbn_tune_step_host_begin(blk.desc, *ins, *outs, arena)
    blk, ins, outs, arena, _ = layers[0]
    C.convbn_tune_step_host_begin(blk.desc, *ins, *outs, arena)      # the same arena again, nothing joined yet
    C.convbn_tune_step_host_join()
    torch.cuda.synchronize()
    C.convbn_check()
    for blk, _, outs, _, want in layers:
        for o, w in zip(outs, want):
            assert (o is None) == (w is None)
            if o is not None:
                assert torch.equal(o, w), blk.spec.name
    C.convbn_tune_step_host_join()                                   # nothing pending: a no-op
