"""Linear-BN (Sec. 3.2.2): pins of the plain numpy definition, and the CUDA path through the 1x1 descriptor."""
import numpy as np
import pytest

from oracle import linear_oracle as LO
from oracle import oracle as O

RNG = np.random.default_rng(11)


def _draw(rows, cin, cout, bias=True):
    return dict(x=RNG.standard_normal((rows, cin)), w=RNG.standard_normal((cout, cin)) * np.sqrt(2.0 / cin),
                b=RNG.standard_normal(cout) * 0.01 if bias else None, gamma=RNG.uniform(0.5, 1.5, cout),
                beta=RNG.standard_normal(cout) * 0.1, mu_hat=RNG.standard_normal(cout) * 0.1,
                var_hat=RNG.uniform(0.5, 2.0, cout))


def test_linear_tune_equals_eval_form_and_the_1x1_convolution_oracle():
    """Two routes that share nothing with the matmul formulas: the Eval form of Sec. 3.1 and the direct-loop
    convolution oracle on rows x 1 x 1 images."""
    t = _draw(13, 7, 5)
    eps = 1e-5
    fw = LO.tune_forward(eps=eps, **t)
    np.testing.assert_allclose(fw["z"], LO.eval_forward(eps=eps, **t), rtol=1e-12, atol=1e-12)
    s = O.Shape(13, 7, 1, 1, 5, 1, 1, eps=eps)
    p = dict(gamma=t["gamma"], beta=t["beta"], mu_hat=t["mu_hat"], var_hat=t["var_hat"])
    cf = O.tune_forward(s, t["x"].reshape(13, 7, 1, 1), t["w"].reshape(5, 7, 1, 1), t["b"], **p)
    np.testing.assert_allclose(fw["z"], cf["z"].reshape(13, 5), rtol=1e-12, atol=1e-12)
    dz = RNG.standard_normal((13, 5))
    bw = LO.tune_backward(dz, t["x"], t["w"], t["b"], t["gamma"], t["mu_hat"], t["var_hat"], eps)
    cb = O.tune_backward(s, dz.reshape(13, 5, 1, 1), t["x"].reshape(13, 7, 1, 1), t["w"].reshape(5, 7, 1, 1), cf["w_f"],
                         t["b"], t["gamma"], t["mu_hat"], t["var_hat"])
    for k in ("dx", "dw", "db", "dgamma", "dbeta"):
        np.testing.assert_allclose(bw[k].ravel(), np.asarray(cb[k]).ravel(), rtol=1e-11, atol=1e-12, err_msg=k)


def test_linear_gradients_match_finite_differences():
    t = _draw(6, 4, 3)
    eps, dz = 1e-5, RNG.standard_normal((6, 3))
    J = lambda: float((dz * LO.tune_forward(eps=eps, **t)["z"]).sum())
    bw = LO.tune_backward(dz, t["x"], t["w"], t["b"], t["gamma"], t["mu_hat"], t["var_hat"], eps)
    for name, grad in (("x", "dx"), ("w", "dw"), ("b", "db"), ("gamma", "dgamma"), ("beta", "dbeta")):
        a = t[name]
        num = np.zeros_like(a)
        for idx in np.ndindex(a.shape):
            keep = a[idx]
            a[idx] = keep + 1e-3; up = J()
            a[idx] = keep - 1e-3; dn = J()
            a[idx] = keep
            num[idx] = (up - dn) / 2e-3
        np.testing.assert_allclose(bw[grad], num, rtol=1e-7, atol=1e-8, err_msg=name)     # Z is linear in each argument


@pytest.mark.gpu
@pytest.mark.parametrize("rows,cin,cout,dtype,bias", [(777, 256, 64, "bf16", False), (1000, 64, 256, "bf16", False),
                                                      (300, 512, 192, "bf16", True), (37, 24, 10, "f32", True),
                                                      (777, 256, 64, "f16", True), (37, 24, 10, "f16", False)])
def test_linear_bn_on_the_device(rows, cin, cout, dtype, bias):
    import torch
    import parity
    from paper_2305_11624_b200 import convbn as C
    from paper_2305_11624_b200 import inputs as I
    tol = parity.TOL[dtype]
    t = _draw(rows, cin, cout, bias)
    rnd = {"bf16": I.round_bf16, "f16": lambda a: np.asarray(a, np.float16).astype(np.float32),
           "f32": lambda a: np.asarray(a, np.float32)}[dtype]
    dz = RNG.standard_normal((rows, cout))
    t["x"], t["w"], dz = (rnd(a.astype(np.float32)).astype(np.float64) for a in (t["x"], t["w"], dz))
    for k in ("b", "gamma", "beta", "mu_hat", "var_hat"):
        if t[k] is not None:
            t[k] = t[k].astype(np.float32).astype(np.float64)
    desc = C.convbn_linear_desc(rows, cin, cout, {"bf16": C.BF16, "f16": C.F16, "f32": C.F32}[dtype], 1e-5)
    td = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    dev = lambda a, d=td: None if a is None else torch.tensor(np.asarray(a, np.float32), device="cuda").to(d).contiguous()
    x, w, dzd = dev(t["x"]), dev(t["w"]), dev(dz)
    vec = {k: dev(t[k], torch.float32) for k in ("b", "gamma", "beta", "mu_hat", "var_hat")}
    z, dx = torch.empty(rows, cout, device="cuda", dtype=td), torch.empty(rows, cin, device="cuda", dtype=td)
    dw = torch.empty(cout, cin, device="cuda")
    db = torch.empty(cout, device="cuda") if bias else None
    dg, dbt = torch.empty(cout, device="cuda"), torch.empty(cout, device="cuda")
    saved = torch.empty(max(16, C.convbn_saved_bytes(desc, C.MODE_TUNE)), dtype=torch.uint8, device="cuda")
    ws = torch.empty(max(256, max(C.convbn_workspace_bytes(desc, p) for p in (C.PHASE_TUNE_FWD, C.PHASE_TUNE_BWD))),
                     dtype=torch.uint8, device="cuda")
    C.convbn_tune_fwd(desc, x, w, vec["b"], vec["gamma"], vec["beta"], vec["mu_hat"], vec["var_hat"], z, saved, ws)
    C.convbn_tune_bwd(desc, dzd, x, w, vec["b"], vec["mu_hat"], saved, dx, dw, db, dg, dbt, ws)
    C.convbn_check()
    fw = LO.tune_forward(eps=1e-5, **t)
    bw = LO.tune_backward(dz, t["x"], t["w"], t["b"], t["gamma"], t["mu_hat"], t["var_hat"], 1e-5)
    host = lambda a: None if a is None else a.float().cpu().numpy().astype(np.float64)
    got = {"z": host(z), "dx": host(dx), "dw": host(dw), "db": host(db), "dgamma": host(dg), "dbeta": host(dbt)}
    ref = dict(bw, z=fw["z"])
    for k in ("z", "dx", "dw", "db", "dgamma", "dbeta"):
        if ref[k] is None:
            continue
        err = O.rel_l2(got[k], ref[k])
        assert err <= tol, (k, err)
