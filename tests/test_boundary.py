"""Host-side contract of the C ABI: the library loads without a GPU, exports every symbol the
header declares, computes shapes and sizes, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as G
from paper_2305_11624_b200 import convbn as C

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    G.build()


def good(**kw):
    base = dict(n=2, c_in=16, h_in=16, w_in=16, c_out=32, kh=3, kw=3, pad_h=1, pad_w=1,
                dtype=C.F32, layout=C.NCHW)
    base.update(kw)
    return C.Desc.make(**base)


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "convbn.h")).read()
    declared = set(re.findall(r"\b(convbn_[a-z_]+)\s*\(", header))
    assert declared == set(C.EXPORTS)
    lib = C.lib()
    for name in declared:
        assert getattr(lib, name) is not None


def test_out_shape_and_sizes():
    assert C.convbn_out_shape(good()) == (16, 16)
    assert C.convbn_out_shape(good(h_in=224, w_in=224, kh=7, kw=7, stride_h=2, stride_w=2, pad_h=3, pad_w=3)) == (112, 112)
    assert C.convbn_out_shape(good(h_in=200, w_in=334, stride_h=2, stride_w=2)) == (100, 167)
    assert C.convbn_out_shape(good(h_in=9, w_in=9, dil_h=2, dil_w=2, pad_h=0, pad_w=0)) == (5, 5)
    d = good()
    assert C.convbn_saved_bytes(d, C.MODE_TUNE) == 3 * 32 * 4          # s, b', r: no feature map
    assert C.convbn_saved_bytes(d, C.MODE_EVAL) == 2 * 32 * 16 * 16 * 4  # the pre-normalisation Y
    assert C.convbn_saved_bytes(d, C.MODE_DEPLOY) == 0
    b = good(dtype=C.BF16, layout=C.NHWC)
    assert C.convbn_saved_bytes(b, C.MODE_EVAL) == 2 * 32 * 16 * 16 * 2
    for ph in range(7):
        assert C.convbn_workspace_bytes(d, ph) % 256 == 0
    assert C.convbn_workspace_bytes(d, C.PHASE_TUNE_FWD) >= 32 * 16 * 9 * 4
    assert C.convbn_workspace_bytes(d, 99) == 0


def test_workspace_sizes_of_the_benchmark_layers():
    """Every phase of every benchmark layer asks for a 256-byte multiple; the parameter-gradient scratch
    (partial tiles per pixel slice) stays within a few tens of MiB, and that of the headline configuration's
    layers within the 16 MiB of the no-allocation entry point."""
    from paper_2305_11624_b200 import inputs as I
    from paper_2305_11624_b200.harness import make_desc
    for ci, layers in I.CONFIGS.items():
        for sp in layers:
            d = make_desc(sp)
            for ph in (C.PHASE_TUNE_FWD, C.PHASE_TUNE_BWD_DATA, C.PHASE_TUNE_BWD_WEIGHT):
                ws = C.convbn_workspace_bytes(d, ph)
                assert ws % 256 == 0 and ws < 64 << 20, (sp.name, ph, ws)
            wsw = C.convbn_workspace_bytes(d, C.PHASE_TUNE_BWD_WEIGHT)
            assert wsw > 0, sp.name
            if ci == 1:
                assert wsw <= 16 << 20, (sp.name, wsw)


@pytest.mark.parametrize("kw", [
    dict(n=0), dict(c_in=-1), dict(kh=0), dict(stride_h=0), dict(dil_w=0), dict(pad_h=-1),
    dict(groups=3), dict(groups=0), dict(h_in=1, w_in=1, pad_h=0, pad_w=0), dict(dtype=7),
    dict(layout=5), dict(eps=-1.0),
])
def test_bad_descriptors_are_rejected_on_the_host(kw):
    d = good(**kw)
    ho, wo = ctypes.c_int(), ctypes.c_int()
    assert C.lib().convbn_out_shape(ctypes.byref(d), ctypes.byref(ho), ctypes.byref(wo)) == C.EINVAL
    assert C.convbn_saved_bytes(d, C.MODE_EVAL) == 0
    assert C.convbn_workspace_bytes(d, C.PHASE_TUNE_FWD) == 0
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tune_fwd(d, 256, 256, None, 256, 256, 256, 256, 256, 256, 256, 1 << 30, stream=0)
    assert e.value.status == C.EINVAL


def test_largest_problems():
    """The documented size limits: 2^40 elements per tensor, 2^30 weights per output channel.  One element below is
    accepted (sizes come back, nothing overflows into a small or negative number), one above is CONVBN_EINVAL."""
    ho, wo = ctypes.c_int(), ctypes.c_int()
    shape = lambda d: C.lib().convbn_out_shape(ctypes.byref(d), ctypes.byref(ho), ctypes.byref(wo))
    one = dict(kh=1, kw=1, pad_h=0, pad_w=0, dtype=C.BF16, layout=C.NHWC)
    # 2^40 activation elements exactly: 2^15 images of 2^7 x 2^8 pixels and 2^10 channels
    at_limit = good(n=1 << 15, c_in=1 << 10, h_in=1 << 7, w_in=1 << 8, c_out=1 << 10, **one)
    assert shape(at_limit) == C.OK and (ho.value, wo.value) == (1 << 7, 1 << 8)
    assert C.convbn_saved_bytes(at_limit, C.MODE_EVAL) == 2 << 40
    assert C.convbn_saved_bytes(at_limit, C.MODE_TUNE) == 3 * 4 * (1 << 10)
    for ph in (C.PHASE_TUNE_FWD, C.PHASE_TUNE_BWD, C.PHASE_EVAL_BWD):
        ws = C.convbn_workspace_bytes(at_limit, ph)
        assert 0 < ws < 3 << 40 and ws % 256 == 0, (ph, ws)      # Eval backward holds dY, a tensor of the size of Z
    assert shape(good(n=(1 << 15) + 1, c_in=1 << 10, h_in=1 << 7, w_in=1 << 8, c_out=1 << 10, **one)) == C.EINVAL   # input
    assert shape(good(n=(1 << 15) + 1, c_in=8, h_in=1 << 7, w_in=1 << 8, c_out=1 << 10, **one)) == C.EINVAL         # output
    # weights per output channel: C_in kh kw <= 2^30
    wide = dict(n=1, h_in=64, w_in=64, c_out=8, pad_h=0, pad_w=0, dtype=C.BF16, layout=C.NHWC)
    assert shape(good(c_in=1 << 18, kh=64, kw=64, **wide)) == C.OK and (ho.value, wo.value) == (1, 1)
    assert shape(good(c_in=(1 << 18) + 8, kh=64, kw=64, **wide)) == C.EINVAL
    # extents that no int holds are rejected, not wrapped
    assert shape(good(n=1, c_in=1, h_in=(1 << 31) - 1, w_in=(1 << 31) - 1, c_out=1, **one)) == C.EINVAL
    assert shape(good(h_in=16, w_in=16, pad_h=(1 << 31) - 1, pad_w=1)) == C.EINVAL


def test_argument_checks_before_any_launch():
    d = good()
    ws = C.convbn_workspace_bytes(d, C.PHASE_TUNE_FWD)
    ok = 4096
    args = lambda **o: {**dict(x=ok, w=ok, b=None, gamma=ok, beta=ok, run_mean=ok, run_var=ok, z=ok,
                               saved=ok, workspace=ok, workspace_bytes=ws, stream=0), **o}

    def status(**o):
        with pytest.raises(C.ConvBNError) as e:
            C.convbn_tune_fwd(d, **args(**o))
        return e.value.status

    assert status(x=None) == C.EINVAL
    assert status(saved=None) == C.EINVAL
    assert status(x=ok + 8) == C.EALIGN
    assert status(gamma=ok + 2) == C.EALIGN
    assert status(workspace=None) == C.EWORKSPACE
    assert status(workspace_bytes=ws - 1) == C.EWORKSPACE
    assert status(workspace=ok + 16) == C.EALIGN
    mixed = good(dtype=C.BF16, layout=C.NCHW)
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tune_fwd(mixed, **args())
    assert e.value.status == C.EUNSUPPORTED
    # db must be given exactly when b is
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tune_bwd_weight(d, ok, ok, ok, ok, ok, ok, ok, None, ok, ok, ok, 1 << 30, stream=0)
    assert e.value.status == C.EINVAL


def test_status_strings():
    assert C.status_string(C.OK) == "ok"
    assert "workspace" in C.status_string(C.EWORKSPACE)
    assert C.status_string(1234) == "unknown status"
    assert C.convbn_last_kernel(99) == "none"
