"""Pins for the fp64 CPU oracle: every check compares it with something that is not the
oracle's own formula - library correlation / matmul, hand-worked delta kernels, brute-force
constructions, exact finite differences, adjoint identities and closed forms."""
import itertools
import os

import numpy as np
import pytest
from scipy.signal import correlate2d

from oracle import oracle as O

RNG = np.random.default_rng(7)


def rnd(*shape):
    return RNG.standard_normal(shape)


def bn_params(c):
    return dict(gamma=RNG.uniform(0.5, 1.5, c), beta=rnd(c) * 0.1, mu_hat=rnd(c) * 0.1,
                var_hat=RNG.uniform(0.5, 2.0, c))


def numpy_bn(y, p, eps):
    """Sec. 3.1 Eval formula retyped with numpy broadcasting (used only on the test side)."""
    v = lambda a: a[None, :, None, None]
    return v(p["gamma"]) * (y - v(p["mu_hat"])) / np.sqrt(v(p["var_hat"]) + eps) + v(p["beta"])


SHAPES = [
    O.Shape(2, 3, 6, 7, 4, 3, 3, pad_h=1, pad_w=1),
    O.Shape(1, 4, 9, 8, 6, 3, 2, stride_h=2, stride_w=1, pad_h=1, pad_w=0),
    O.Shape(2, 4, 10, 9, 4, 3, 3, stride_h=2, stride_w=2, pad_h=1, pad_w=1, groups=2),
    O.Shape(1, 6, 8, 8, 6, 3, 3, pad_h=2, pad_w=2, dil_h=2, dil_w=2, groups=6),
    O.Shape(2, 5, 5, 5, 3, 1, 1),
    O.Shape(1, 2, 11, 12, 3, 5, 3, stride_h=3, stride_w=2, pad_h=2, pad_w=1, dil_h=1, dil_w=2),
]


# ---- forward: library special cases ------------------------------------------------------

@pytest.mark.parametrize("s", SHAPES[:2] + [O.Shape(1, 3, 7, 6, 2, 3, 3, pad_h=2, pad_w=1)])
def test_conv_matches_scipy_correlate_stride1_or_subsampled(s):
    """Plain cross-correlation (no kernel flip): zero-pad, 'valid' correlate2d per channel
    pair, sum over input channels, subsample by the stride."""
    x, w, b = rnd(*s.x_shape), rnd(*s.w_shape), rnd(s.c_out)
    y = O.conv(s, x, w, b)
    xp = np.pad(x, ((0, 0), (0, 0), (s.pad_h, s.pad_h), (s.pad_w, s.pad_w)))
    for n, co in itertools.product(range(s.n), range(s.c_out)):
        full = sum(correlate2d(xp[n, ci], w[co, ci], mode="valid") for ci in range(s.c_in)) + b[co]
        np.testing.assert_allclose(y[n, co], full[::s.stride_h, ::s.stride_w], rtol=1e-12, atol=1e-12)


def test_identity_bn_reduces_block_to_plain_correlation():
    """gamma = sqrt(var+eps), mu = 0, beta = 0, b = 0: Eval, Deploy and Tune all give the bare
    cross-correlation."""
    s = O.Shape(1, 2, 6, 6, 3, 3, 3, pad_h=1, pad_w=1)
    x, w = rnd(*s.x_shape), rnd(*s.w_shape)
    var = RNG.uniform(0.5, 2, s.c_out)
    p = dict(gamma=np.sqrt(var + s.eps), beta=np.zeros(s.c_out), mu_hat=np.zeros(s.c_out), var_hat=var)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    want = np.stack([sum(correlate2d(xp[0, ci], w[co, ci], mode="valid") for ci in range(2))
                     for co in range(3)])[None]
    z_eval = O.eval_forward(s, x, w, None, **p)["z"]
    z_tune = O.tune_forward(s, x, w, None, **p)["z"]
    np.testing.assert_allclose(z_eval, want, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(z_tune, want, rtol=1e-12, atol=1e-12)


def test_pointwise_conv_is_a_matmul():
    s = SHAPES[4]
    x, w, b = rnd(*s.x_shape), rnd(*s.w_shape), rnd(s.c_out)
    want = np.einsum("oc,nchw->nohw", w[:, :, 0, 0], x) + b[None, :, None, None]
    np.testing.assert_allclose(O.conv(s, x, w, b), want, rtol=1e-12, atol=1e-12)


def test_depthwise_is_per_channel_correlation():
    s = O.Shape(2, 5, 7, 6, 5, 3, 3, pad_h=1, pad_w=1, groups=5)
    x, w = rnd(*s.x_shape), rnd(*s.w_shape)
    y = O.conv(s, x, w)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    for n, c in itertools.product(range(2), range(5)):
        np.testing.assert_allclose(y[n, c], correlate2d(xp[n, c], w[c, 0], mode="valid"),
                                   rtol=1e-12, atol=1e-12)


def test_delta_kernels_by_hand():
    """1-channel 3x3 kernels with a single 1: centre tap = identity; tap (r,q) reads
    x[h - pad + r, w - pad + q], so tap (0,0) with pad 1 shifts the image down-right by one and
    fills the first row/column with zeros; stride 2 keeps every other sample; dilation 2 with
    pad 2 and tap (0,0) shifts by two."""
    x = np.arange(1.0, 26.0).reshape(1, 1, 5, 5)
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 1, 1] = 1
    s = O.Shape(1, 1, 5, 5, 1, 3, 3, pad_h=1, pad_w=1)
    np.testing.assert_array_equal(O.conv(s, x, w), x)
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 0] = 1
    want = np.zeros_like(x); want[0, 0, 1:, 1:] = x[0, 0, :-1, :-1]
    np.testing.assert_array_equal(O.conv(s, x, w), want)
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 2, 1] = 1           # reads the row below
    want = np.zeros_like(x); want[0, 0, :-1, :] = x[0, 0, 1:, :]
    np.testing.assert_array_equal(O.conv(s, x, w), want)
    s2 = O.Shape(1, 1, 5, 5, 1, 3, 3, stride_h=2, stride_w=2, pad_h=1, pad_w=1)
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 1, 1] = 1
    np.testing.assert_array_equal(O.conv(s2, x, w), x[:, :, ::2, ::2])
    assert O.out_hw(s2) == (3, 3)
    sd = O.Shape(1, 1, 5, 5, 1, 3, 3, pad_h=2, pad_w=2, dil_h=2, dil_w=2)
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 0] = 1
    want = np.zeros_like(x); want[0, 0, 2:, 2:] = x[0, 0, :-2, :-2]
    np.testing.assert_array_equal(O.conv(sd, x, w), want)


def test_output_sizes_of_known_layers():
    """Output extents fixed by the benchmark configuration text (see tests/golden)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "layer_output_sizes.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 6
    for h_in, w_in, k, stride, pad, h_out, w_out in (map(int, r) for r in rows):
        s = O.Shape(1, 1, h_in, w_in, 1, k, k, stride_h=stride, stride_w=stride, pad_h=pad, pad_w=pad)
        assert O.out_hw(s) == (h_out, w_out)


# ---- forward: brute-force constructions for groups / stride / dilation ----------------------

def test_groups_equal_independent_dense_problems():
    s = SHAPES[2]
    x, w, b = rnd(*s.x_shape), rnd(*s.w_shape), rnd(s.c_out)
    y = O.conv(s, x, w, b)
    cg, cog = s.c_in // s.groups, s.c_out // s.groups
    for g in range(s.groups):
        sg = O.Shape(s.n, cg, s.h_in, s.w_in, cog, s.kh, s.kw, s.stride_h, s.stride_w, s.pad_h,
                     s.pad_w, s.dil_h, s.dil_w, 1)
        yg = O.conv(sg, x[:, g * cg:(g + 1) * cg], w[g * cog:(g + 1) * cog], b[g * cog:(g + 1) * cog])
        np.testing.assert_allclose(y[:, g * cog:(g + 1) * cog], yg, rtol=1e-13, atol=1e-13)


def test_dilation_equals_zero_stuffed_kernel():
    s = O.Shape(1, 2, 9, 10, 3, 3, 2, pad_h=2, pad_w=1, dil_h=2, dil_w=3)
    x, w = rnd(*s.x_shape), rnd(*s.w_shape)
    eh, ew = s.dil_h * (s.kh - 1) + 1, s.dil_w * (s.kw - 1) + 1
    wz = np.zeros((s.c_out, s.c_in, eh, ew)); wz[:, :, ::s.dil_h, ::s.dil_w] = w
    sz = O.Shape(1, 2, 9, 10, 3, eh, ew, pad_h=2, pad_w=1)
    np.testing.assert_allclose(O.conv(s, x, w), O.conv(sz, x, wz), rtol=1e-13, atol=1e-13)


# ---- the paper's equivalences ---------------------------------------------------------------

@pytest.mark.parametrize("s", SHAPES)
@pytest.mark.parametrize("bias", [True, False])
def test_eval_deploy_tune_forward_agree(s, bias):
    """Sec. 3.3: Eval and Deploy give equivalent forward results; Sec. 3.4: so does Tune.  The
    Eval route is also compared with the Sec. 3.1 formula retyped in numpy."""
    x, w = rnd(*s.x_shape), rnd(*s.w_shape)
    b = rnd(s.c_out) if bias else None
    p = bn_params(s.c_out)
    ev = O.eval_forward(s, x, w, b, **p)
    tu = O.tune_forward(s, x, w, b, **p)
    dep = O.deploy_forward(s, x, *O.fold(s, w, b, **p))
    np.testing.assert_allclose(ev["z"], numpy_bn(ev["y"], p, s.eps), rtol=1e-12, atol=1e-12)
    assert O.rel_l2(tu["z"], ev["z"]) < 1e-13
    assert O.rel_l2(dep, ev["z"]) < 1e-13
    sc = p["gamma"] / np.sqrt(p["var_hat"] + s.eps)
    np.testing.assert_allclose(tu["w_f"], w * sc[:, None, None, None], rtol=1e-14)
    np.testing.assert_allclose(tu["b_f"], ((0 if b is None else b) - p["mu_hat"]) * sc + p["beta"], rtol=1e-13)


def _J(s, dz, x, w, b, p):
    """J = <dZ, Z_eval(x, w, b, gamma, beta)> through the Eval route (conv, then BN)."""
    return float(np.sum(dz * O.eval_forward(s, x, w, b, **p)["z"]))


def _fd(f, a, h=1e-3):
    """Central differences of scalar f over every element of a (exact for f linear in a)."""
    g = np.empty_like(a)
    it = np.nditer(a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = a[i]
        a[i] = old + h; fp = f()
        a[i] = old - h; fm = f()
        a[i] = old
        g[i] = (fp - fm) / (2 * h)
    return g


FD_SHAPES = [
    O.Shape(2, 2, 4, 5, 3, 3, 3, pad_h=1, pad_w=1),
    O.Shape(1, 4, 6, 5, 4, 3, 2, stride_h=2, stride_w=1, pad_h=1, pad_w=1, dil_h=1, dil_w=2, groups=2),
    O.Shape(1, 3, 5, 5, 3, 3, 3, stride_h=2, stride_w=2, pad_h=1, pad_w=1, groups=3),
]


@pytest.mark.parametrize("s", FD_SHAPES)
@pytest.mark.parametrize("route", ["tune", "eval"])
@pytest.mark.parametrize("bias", [True, False])
def test_all_gradients_match_finite_differences(s, route, bias):
    """Z is linear in each of X, omega, b, gamma, beta separately, so central differences of
    J = <dZ, Z> are exact up to rounding: a tight pin on all five gradients of both the
    Tune-row and the Eval-row equations of Table 2."""
    x, w, dz = rnd(*s.x_shape), rnd(*s.w_shape), rnd(*s.z_shape)
    b = rnd(s.c_out) if bias else None
    p = bn_params(s.c_out)
    if route == "tune":
        w_f = O.tune_forward(s, x, w, b, **p)["w_f"]
        g = O.tune_backward(s, dz, x, w, w_f, b, p["gamma"], p["mu_hat"], p["var_hat"])
    else:
        y = O.eval_forward(s, x, w, b, **p)["y"]
        g = O.eval_backward(s, dz, x, y, w, p["gamma"], p["mu_hat"], p["var_hat"], with_bias=bias)
    f = lambda: _J(s, dz, x, w, b, p)
    tol = dict(rtol=1e-8, atol=1e-8)
    np.testing.assert_allclose(g["dx"], _fd(f, x), **tol)
    np.testing.assert_allclose(g["dw"], _fd(f, w), **tol)
    np.testing.assert_allclose(g["dgamma"], _fd(f, p["gamma"]), **tol)
    np.testing.assert_allclose(g["dbeta"], _fd(f, p["beta"]), **tol)
    if bias:
        np.testing.assert_allclose(g["db"], _fd(f, b), **tol)
    else:
        assert g["db"] is None


@pytest.mark.parametrize("s", SHAPES)
def test_adjoint_identities(s):
    """<omega (*) X, dY> = <X, dX> = <omega, domega> (Sec. 3.2.1 gradients are the adjoints of
    the bilinear forward map)."""
    x, w, dy = rnd(*s.x_shape), rnd(*s.w_shape), rnd(*s.z_shape)
    lhs = float(np.sum(O.conv(s, x, w) * dy))
    assert abs(float(np.sum(x * O.conv_grad_input(s, dy, w))) - lhs) <= 1e-11 * max(1, abs(lhs))
    assert abs(float(np.sum(w * O.conv_grad_weight(s, dy, x))) - lhs) <= 1e-11 * max(1, abs(lhs))


def test_grad_input_stride1_is_correlation_with_rotated_kernel():
    """dX = omega_rot (*) dY: for stride 1 this is the 'full' cross-correlation of dY with the
    180-degree rotated kernel, summed over output channels, cropped by the padding."""
    s = O.Shape(1, 2, 6, 7, 3, 3, 3, pad_h=1, pad_w=1)
    w, dy = rnd(*s.w_shape), rnd(*s.z_shape)
    dx = O.conv_grad_input(s, dy, w)
    for ci in range(s.c_in):
        full = sum(correlate2d(dy[0, co], w[co, ci, ::-1, ::-1], mode="full") for co in range(s.c_out))
        np.testing.assert_allclose(dx[0, ci], full[1:-1, 1:-1], rtol=1e-12, atol=1e-12)


def test_grad_weight_stride1_is_correlation_of_input_with_dy():
    s = O.Shape(2, 2, 6, 7, 3, 3, 3, pad_h=1, pad_w=1)
    x, dy = rnd(*s.x_shape), rnd(*s.z_shape)
    dw = O.conv_grad_weight(s, dy, x)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    for co, ci in itertools.product(range(3), range(2)):
        want = sum(correlate2d(xp[n, ci], dy[n, co], mode="valid") for n in range(2))
        np.testing.assert_allclose(dw[co, ci], want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("s", SHAPES)
def test_tune_and_eval_backward_agree_and_closed_forms(s):
    """Sec. 3.4: equal forward maps of (omega, b, gamma, beta) have equal Jacobians, so the
    Tune-row and Eval-row equations must give the same five gradients; dbeta = sum dZ and
    db = s sum dZ in closed form (Table 2, Appendix B)."""
    x, w, dz, b = rnd(*s.x_shape), rnd(*s.w_shape), rnd(*s.z_shape), rnd(s.c_out)
    p = bn_params(s.c_out)
    ev = O.eval_forward(s, x, w, b, **p)
    tu = O.tune_forward(s, x, w, b, **p)
    ge = O.eval_backward(s, dz, x, ev["y"], w, p["gamma"], p["mu_hat"], p["var_hat"])
    gt = O.tune_backward(s, dz, x, w, tu["w_f"], b, p["gamma"], p["mu_hat"], p["var_hat"])
    for k in ("dx", "dw", "db", "dgamma", "dbeta"):
        assert O.rel_l2(gt[k], ge[k]) < 1e-12, k
    sums = dz.sum(axis=(0, 2, 3))
    sc = p["gamma"] / np.sqrt(p["var_hat"] + s.eps)
    np.testing.assert_allclose(gt["dbeta"], sums, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gt["db"], sc * sums, rtol=1e-12, atol=1e-12)
    gd = O.deploy_backward(s, dz, x, tu["w_f"])
    assert O.rel_l2(gd["dx"], gt["dx"]) < 1e-13
    np.testing.assert_allclose(gd["dw_f"] * sc[:, None, None, None], gt["dw"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gd["db_f"], sums, rtol=1e-12, atol=1e-12)


def test_planted_mistakes_are_caught():
    """The pins must be able to fail: a kernel flip, a dropped dgamma term and a missing s in
    domega each break the finite-difference or library comparison."""
    s = O.Shape(1, 2, 5, 5, 2, 3, 3, pad_h=1, pad_w=1)
    x, w, dz, b = rnd(*s.x_shape), rnd(*s.w_shape), rnd(*s.z_shape), rnd(s.c_out)
    p = bn_params(s.c_out)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    flipped = O.conv(s, x, w[:, :, ::-1, ::-1])
    want = sum(correlate2d(xp[0, ci], w[0, ci], mode="valid") for ci in range(2))
    assert not np.allclose(flipped[0, 0], want)
    w_f = O.tune_forward(s, x, w, b, **p)["w_f"]
    g = O.tune_backward(s, dz, x, w, w_f, b, p["gamma"], p["mu_hat"], p["var_hat"])
    fd_gamma = _fd(lambda: _J(s, dz, x, w, b, p), p["gamma"])
    r = 1 / np.sqrt(p["var_hat"] + s.eps)
    dropped = g["dgamma"] - g["dbeta"] * (b - p["mu_hat"]) * r
    assert not np.allclose(dropped, fd_gamma, rtol=1e-6)
    unscaled = O.conv_grad_weight(s, dz, x)
    assert not np.allclose(unscaled, _fd(lambda: _J(s, dz, x, w, b, p), w), rtol=1e-6)


def test_saved_elements_follow_appendix_m():
    """Appendix M memory analysis: Eval keeps X + Y, Tune X + omega', Deploy X; the saving
    N C_out H_out W_out - k^2 C_in C_out is negative for the 3x3 512->512 layer at 7x7, N=64."""
    s = O.Shape(32, 64, 56, 56, 64, 3, 3, pad_h=1, pad_w=1)
    assert O.saved_elements(s, "eval") == 2 * 32 * 64 * 56 * 56
    assert O.saved_elements(s, "tune") == 32 * 64 * 56 * 56 + 9 * 64 * 64
    assert O.saved_elements(s, "deploy") == 32 * 64 * 56 * 56
    t = O.Shape(64, 512, 7, 7, 512, 3, 3, pad_h=1, pad_w=1)
    assert O.saved_elements(t, "eval") - O.saved_elements(t, "tune") == 64 * 512 * 49 - 9 * 512 * 512 < 0


# ---- the comparator and the per-channel scale: hand values ---------------------------------

def test_rel_l2_on_hand_values():
    """The norm behind every parity verdict: ||got - ref|| / ||ref||, absolute when ref = 0."""
    assert O.rel_l2([1.0, 0.0], [0.0, 1.0]) == pytest.approx(np.sqrt(2.0), rel=1e-15)
    assert O.rel_l2([3.0, 4.0], [0.0, 0.0]) == 5.0              # zero reference: absolute norm
    x = rnd(37)
    assert O.rel_l2(x, x) == 0.0
    assert O.rel_l2([2.0, 0.0, 0.0], [1.0, 0.0, 0.0]) == 1.0    # 100 % error on the only non-zero entry
    assert O.rel_l2([[1.0, 2.0], [3.0, 5.0]], [[1.0, 2.0], [3.0, 4.0]]) == pytest.approx(1.0 / np.sqrt(30.0), rel=1e-15)
    # a sign flip of the whole tensor is an error of 2, a transposed operand is seen
    assert O.rel_l2(-x, x) == pytest.approx(2.0, rel=1e-15)
    a = np.array([[1.0, 2.0], [3.0, 4.0]])
    assert O.rel_l2(a.T, a) > 0.1


def test_scale_on_hand_values():
    """Sec. 3.3: r = 1 / sqrt(var_hat + eps), s = gamma r, with eps INSIDE the root."""
    s = O.Shape(1, 1, 1, 1, 3, 1, 1, eps=1.0)
    sc, r = O.scale(s, gamma=[3.0, -2.0, 0.5], var_hat=[15.0, 3.0, 0.0])
    np.testing.assert_allclose(r, [0.25, 0.5, 1.0], rtol=1e-15)
    np.testing.assert_allclose(sc, [0.75, -1.0, 0.5], rtol=1e-15)
    # the same s folds the weights: omega' = s omega, b' = (b - mu) s + beta on a 1x1 block
    w = np.array([2.0, 4.0, 8.0]).reshape(3, 1, 1, 1)
    w_f, b_f = O.fold(s, w, np.array([1.0, 1.0, 1.0]), gamma=[3.0, -2.0, 0.5], beta=[0.5, 0.5, 0.5],
                      mu_hat=[3.0, 0.0, -1.0], var_hat=[15.0, 3.0, 0.0])
    np.testing.assert_allclose(w_f.ravel(), [1.5, -4.0, 4.0], rtol=1e-15)
    np.testing.assert_allclose(b_f, [(1 - 3) * 0.75 + 0.5, -1.0 + 0.5, 2 * 0.5 + 0.5], rtol=1e-15)
