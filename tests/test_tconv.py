"""TransposedConv-BN in Tune mode: pins of the numpy oracle (CPU) and parity of the library against it (GPU)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from oracle import tconv_oracle as T

CASES = [  # (n, c_in, h, w, c_out, k, stride, pad, dil, groups)
    (2, 3, 4, 5, 4, 3, 1, 0, 1, 1),
    (1, 4, 5, 4, 6, 2, 2, 0, 1, 1),       # the U-Net up-sampling shape: kernel = stride
    (2, 4, 3, 4, 2, 3, 2, 1, 1, 2),
    (1, 2, 4, 3, 3, 4, 2, 1, 1, 1),       # kernel 4, stride 2, pad 1: doubles the extent
    (1, 2, 3, 3, 2, 3, 1, 2, 2, 1),
]


def _rnd(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


def _params(seed, c):
    g = np.random.default_rng(seed)
    return dict(gamma=g.uniform(0.5, 1.5, c), beta=g.normal(0, 0.1, c), mu_hat=g.normal(0, 0.1, c), var_hat=g.uniform(0.5, 2.0, c))


def _make(case, seed=0):
    n, ci, h, w, co, k, st, pad, dil, grp = case
    x, wt, b = _rnd(seed, n, ci, h, w), _rnd(seed + 1, ci, co // grp, k, k), _rnd(seed + 2, co)
    ho, wo = T.out_hw(h, w, k, k, st, pad, dil)
    return x, wt, b, _params(seed + 3, co), _rnd(seed + 4, n, co, ho, wo), dict(stride=st, pad=pad, dil=dil, groups=grp)


def test_scatter_by_hand():
    """One input pixel of value 1 copies the kernel (no flip) to the output; stride 2 with a 2x2 kernel of ones
    replicates every input pixel into a 2x2 block."""
    k = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(1, 1, 2, 2)
    x = np.zeros((1, 1, 2, 2)); x[0, 0, 0, 0] = 1.0
    out = T.conv_transpose(x, k)
    assert out.shape == (1, 1, 3, 3)
    np.testing.assert_array_equal(out[0, 0], [[1, 2, 0], [3, 4, 0], [0, 0, 0]])
    x = np.arange(4.0).reshape(1, 1, 2, 2)
    up = T.conv_transpose(x, np.ones((1, 1, 2, 2)), stride=2)
    np.testing.assert_array_equal(up[0, 0], np.kron(x[0, 0], np.ones((2, 2))))
    # padding crops the border, dilation spreads the taps
    np.testing.assert_array_equal(T.conv_transpose(x, k, pad=1)[0, 0], [[0 * 4 + 1 * 3 + 2 * 2 + 3 * 1]])
    d = T.conv_transpose(np.ones((1, 1, 1, 1)), k, dil=2)[0, 0]
    np.testing.assert_array_equal(d, [[1, 0, 2], [0, 0, 0], [3, 0, 4]])


@pytest.mark.parametrize("case", CASES)
def test_transposed_convolution_is_the_adjoint_of_the_pinned_convolution(case):
    n, ci, h, w, co, k, st, pad, dil, grp = case
    x, wt, *_ = _make(case)
    ho, wo = T.out_hw(h, w, k, k, st, pad, dil)
    s = O.Shape(n, co, ho, wo, ci, k, k, st, st, pad, pad, dil, dil, grp)     # the convolution it transposes
    assert O.out_hw(s) == (h, w)
    got = T.conv_transpose(x, wt, st, pad, dil, grp)
    np.testing.assert_allclose(got, O.conv_grad_input(s, x, wt), rtol=1e-12, atol=1e-12)
    y = _rnd(9, n, co, ho, wo)
    assert np.vdot(got, y) == pytest.approx(np.vdot(x, O.conv(s, y, wt)), rel=1e-12)


@pytest.mark.parametrize("case", CASES)
def test_matches_the_library_routine(case):
    n, ci, h, w, co, k, st, pad, dil, grp = case
    x, wt, *_ = _make(case)
    ref = torch.nn.functional.conv_transpose2d(torch.from_numpy(x), torch.from_numpy(wt), stride=st, padding=pad,
                                               dilation=dil, groups=grp).numpy()
    np.testing.assert_allclose(T.conv_transpose(x, wt, st, pad, dil, grp), ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("case", CASES)
def test_tune_form_equals_eval_form(case):
    x, wt, b, p, _, kw = _make(case)
    for bias in (b, None):
        tune = T.tune_forward(x, wt, bias, eps=1e-5, **p, **kw)["z"]
        np.testing.assert_allclose(tune, T.eval_forward(x, wt, bias, eps=1e-5, **p, **kw), rtol=1e-12, atol=1e-12)


def test_scale_and_fold_on_hand_values():
    s, r = T.scale([3.0, -2.0], [15.0, 3.0], 1.0)
    np.testing.assert_allclose(r, [0.25, 0.5]); np.testing.assert_allclose(s, [0.75, -1.0])
    # the scale follows the OUTPUT channel, the second weight axis: w [C_in = 2][C_out = 2][1][1]
    w = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(2, 2, 1, 1)
    w_f, b_f = T.fold(w, np.array([1.0, 1.0]), [3.0, -2.0], [0.5, 0.5], [3.0, 0.0], [15.0, 3.0], 1.0)
    np.testing.assert_allclose(w_f.reshape(2, 2), [[0.75, -2.0], [2.25, -4.0]])
    np.testing.assert_allclose(b_f, [(1 - 3) * 0.75 + 0.5, -1.0 + 0.5])
    # with two groups, input channel 1 feeds output channel 1: w [2][1][1][1]
    w_f, _ = T.fold(np.array([5.0, 7.0]).reshape(2, 1, 1, 1), None, [3.0, -2.0], [0, 0], [0, 0], [15.0, 3.0], 1.0, groups=2)
    np.testing.assert_allclose(w_f.ravel(), [3.75, -7.0])


@pytest.mark.parametrize("case", CASES)
def test_gradients_match_finite_differences(case):
    """J = <dZ, Z> is linear in each of x, w, b, gamma, beta: central differences are exact to rounding."""
    x, wt, b, p, dz, kw = _make(case)
    g = T.tune_backward(dz, x, wt, b, p["gamma"], p["mu_hat"], p["var_hat"], 1e-5, **kw)
    J = lambda: float(np.vdot(dz, T.tune_forward(x, wt, b, eps=1e-5, **p, **kw)["z"]))

    def fd(arr):
        out, h = np.zeros_like(arr), 1e-3
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            keep = arr[i]
            arr[i] = keep + h; jp = J()
            arr[i] = keep - h; jm = J()
            arr[i] = keep
            out[i] = (jp - jm) / (2 * h)
        return out

    for name, arr in (("dx", x), ("dw", wt), ("db", b), ("dgamma", p["gamma"]), ("dbeta", p["beta"])):
        np.testing.assert_allclose(g[name], fd(arr), rtol=1e-7, atol=1e-8, err_msg=name)
    # closed forms
    np.testing.assert_allclose(g["dbeta"], dz.sum(axis=(0, 2, 3)))
    s, _ = T.scale(p["gamma"], p["var_hat"], 1e-5)
    np.testing.assert_allclose(g["db"], s * g["dbeta"])


# ---- the library against the oracle ----------------------------------------------------------------------------
GPU_CASES = [  # (dtype, n, c_in, h, w, c_out, k, stride, pad, dil, groups, bias)
    ("f32", 2, 3, 4, 5, 4, 3, 1, 0, 1, 1, True),
    ("f32", 1, 4, 5, 4, 6, 2, 2, 0, 1, 1, True),
    ("f32", 2, 4, 3, 4, 2, 3, 2, 1, 1, 2, False),
    ("f32", 1, 2, 3, 3, 2, 3, 1, 2, 2, 1, True),
    ("bf16", 2, 128, 28, 28, 64, 2, 2, 0, 1, 1, False),     # U-Net up-sampling: kernel = stride = 2
    ("bf16", 2, 64, 16, 20, 64, 4, 2, 1, 1, 1, True),       # kernel 4, stride 2, pad 1
    ("bf16", 2, 64, 30, 30, 128, 3, 1, 1, 1, 1, False),     # stride 1: the strip kernel on both passes
    ("bf16", 3, 64, 9, 11, 64, 3, 2, 1, 1, 2, True),        # two groups, ragged extent
    ("bf16", 1, 256, 56, 56, 128, 2, 2, 0, 1, 1, False),    # several tiles per CTA
    ("f16", 2, 128, 28, 28, 64, 2, 2, 0, 1, 1, True),       # IEEE half: up-sampling, stride 1, and the direct kernels
    ("f16", 2, 64, 30, 30, 128, 3, 1, 1, 1, 1, False),
    ("f16", 2, 12, 9, 11, 20, 3, 2, 1, 1, 2, True),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", GPU_CASES, ids=lambda c: "%s_c%d_%dx%d_o%d_k%d_s%d_g%d" % (c[0], c[2], c[3], c[4], c[5], c[6], c[7], c[10]))
def test_library_matches_the_oracle(case):
    import parity
    from paper_2305_11624_b200 import convbn as C
    from paper_2305_11624_b200 import inputs as I
    dtype, n, ci, h, w, co, k, st, pad, dil, grp, bias = case
    bf = dtype in ("bf16", "f16")           # 16-bit storage, NHWC
    lay = "nhwc" if bf else "nchw"
    rnd = {"bf16": lambda a: I.round_bf16(a.astype(np.float32)).astype(np.float64),
           "f16": lambda a: a.astype(np.float16).astype(np.float64),
           "f32": lambda a: a.astype(np.float32).astype(np.float64)}[dtype]
    x = rnd(_rnd(1, n, ci, h, w))
    wt = rnd(_rnd(2, ci, co // grp, k, k) * np.sqrt(2.0 / (ci // grp * k * k)))
    ho, wo = T.out_hw(h, w, k, k, st, pad, dil)
    dz = rnd(_rnd(3, n, co, ho, wo))
    f32 = lambda a: a.astype(np.float32).astype(np.float64)
    p = {key: f32(val) for key, val in _params(4, co).items()}
    b = f32(_rnd(5, co) * 0.01) if bias else None
    kw = dict(stride=st, pad=pad, dil=dil, groups=grp)
    ref = T.tune_forward(x, wt, b, eps=1e-5, **p, **kw)
    ref.update(T.tune_backward(dz, x, wt, b, p["gamma"], p["mu_hat"], p["var_hat"], 1e-5, **kw))

    dev = "cuda:0"
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    up = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).reshape(-1).to(dt).to(dev)
    desc = C.Desc.make(n, ci, h, w, co, k, k, st, st, pad, pad, dil, dil, grp, {"bf16": C.BF16, "f16": C.F16, "f32": C.F32}[dtype], C.NHWC if bf else C.NCHW, 1e-5)
    assert C.convbn_tconv_out_shape(desc) == (ho, wo)
    X, W, DZ = up(I.act_to_layout(x, lay), tdt), up(I.weight_to_layout(wt, lay), tdt), up(I.act_to_layout(dz, lay), tdt)
    G, Bt, M, V = (up(p[key]) for key in ("gamma", "beta", "mu_hat", "var_hat"))
    Bv = up(b) if bias else None
    Z = torch.full((n * co * ho * wo,), float("nan"), dtype=tdt, device=dev)
    DX = torch.full((x.size,), float("nan"), dtype=tdt, device=dev)
    DW = torch.full((wt.size,), float("nan"), device=dev)
    DB = torch.full((co,), float("nan"), device=dev) if bias else None
    DG, DBt = torch.full((co,), float("nan"), device=dev), torch.full((co,), float("nan"), device=dev)
    saved = torch.empty(3 * co, device=dev)
    ws = torch.empty(max(256, C.convbn_tconv_workspace_bytes(desc)), dtype=torch.uint8, device=dev)
    C.convbn_tconv_tune_fwd(desc, X, W, Bv, G, Bt, M, V, Z, saved, ws)
    C.convbn_tconv_tune_bwd(desc, DZ, X, W, Bv, M, saved, DX, DW, DB, DG, DBt, ws)
    C.convbn_check()
    dn = lambda t: t.float().cpu().numpy().astype(np.float64)
    got = {"z": I.act_from_layout(dn(Z), lay, (n, co, ho, wo)), "dx": I.act_from_layout(dn(DX), lay, x.shape),
           "dw": I.weight_from_layout(dn(DW), lay, wt.shape), "dgamma": dn(DG), "dbeta": dn(DBt)}
    if bias:
        got["db"] = dn(DB)
    tol = parity.TOL[dtype]
    errs = {key: O.rel_l2(val, ref[key]) for key, val in got.items()}
    print(errs)
    assert all(np.isfinite(v) and v <= tol for v in errs.values()), errs
    # per element, on the activations (z carries two bf16 roundings: the convolution's and the bias add's)
    for key in ("z", "dx"):
        assert parity.elem_excess(got[key], ref[key], parity.ELEM_BOUND[dtype], channel_axis=1) <= 1.0, key


def test_tconv_symbols_and_argument_checks():
    from paper_2305_11624_b200 import convbn as C
    d = C.Desc.make(1, 8, 4, 4, 8, 3, 3, 2, 2, 1, 1)
    assert C.convbn_tconv_out_shape(d) == (7, 7)
    assert C.convbn_tconv_workspace_bytes(d) > 0
    bad = C.Desc.make(1, 8, 2, 2, 8, 1, 1, 1, 1, 3, 3)          # padding eats the whole output
    with pytest.raises(C.ConvBNError):
        C.convbn_tconv_out_shape(bad)
    assert C.convbn_tconv_workspace_bytes(bad) == 0
    with pytest.raises(C.ConvBNError) as e:                      # NULL pointers are refused before any launch
        C.convbn_tconv_tune_fwd(d, None, None, None, None, None, None, None, None, None, None, 0, stream=0)
    assert e.value.status == C.EINVAL
    ok = 4096                                                    # fake aligned addresses: checks come before any launch
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tconv_tune_fwd(d, ok, ok, None, ok, ok, ok, ok, ok, ok, None, 0, stream=0)
    assert e.value.status == C.EWORKSPACE
    with pytest.raises(C.ConvBNError) as e:
        C.convbn_tconv_tune_bwd(d, ok, ok, ok, ok, ok, ok, ok, ok, None, ok, ok, ok, 1 << 30, stream=0)
    assert e.value.status == C.EINVAL                            # b without db
