"""Pins for the oracle's statements of Eq. 4 (VDN combined with a sampling rule) and of Appendix D
(moving average, validation forward)."""
import numpy as np
import pytest
import torch

import bns_inputs as I
import oracle as O

EPS = 1e-5


def small(seed, N=6, C=4, H=5, W=7, nv=2):
    x = I.tiny_activations(N, C, H, W, seed)
    dy = I.upstream_gradient(x.shape, seed)
    gamma, beta = I.affine_parameters(C, seed)
    xv = I.virtual_samples(nv, C, H, W, seed)
    dyv = I.upstream_gradient(xv.shape, seed, I.TAG_DYV)
    return x, dy, gamma, beta, xv, dyv


def rules(N, C, H, W, seed):
    return {"batch": O.Sampling.batch(np.array([4, 1], np.int32)),
            "feature": O.Sampling.feature(2, 3, I.patch_offsets(N, C, H, W, 2, 3, I.OFFSETS_PER_MAP, seed),
                                          O.OFFSETS_PER_MAP)}


# --------------------------------------------------------------------------- Eq. 4
def test_mixed_statistics_are_eq4_of_numpy_statistics():
    x, dy, gamma, beta, xv, dyv = small(41)
    N, C, H, W = x.shape
    xs = x[[4, 1]].astype(np.float64)
    xvd = xv.astype(np.float64)
    for mix in (0.5, 0.25):
        f = O.forward_mixed(x, xv, gamma, beta, EPS, mix, rules(N, C, H, W, 41)["batch"])
        np.testing.assert_allclose(f.mean_s, xs.mean(axis=(0, 2, 3)), atol=1e-14)
        np.testing.assert_allclose(f.var_s, xs.var(axis=(0, 2, 3)), rtol=1e-13)
        np.testing.assert_allclose(f.mean_v, xvd.mean(axis=(0, 2, 3)), atol=1e-14)
        np.testing.assert_allclose(f.var_v, xvd.var(axis=(0, 2, 3)), rtol=1e-13)
        np.testing.assert_allclose(f.mean, mix * f.mean_v + (1 - mix) * f.mean_s, rtol=1e-15)
        np.testing.assert_allclose(f.var, mix * f.var_v + (1 - mix) * f.var_s, rtol=1e-15)
        sh = (1, -1, 1, 1)
        g, b = gamma.astype(np.float64).reshape(sh), beta.astype(np.float64).reshape(sh)
        want = g * (x.astype(np.float64) - f.mean.reshape(sh)) / np.sqrt(f.var.reshape(sh) + EPS) + b
        np.testing.assert_allclose(f.y, want, rtol=1e-13, atol=1e-14)
        want_v = g * (xvd - f.mean.reshape(sh)) / np.sqrt(f.var.reshape(sh) + EPS) + b
        np.testing.assert_allclose(f.yv, want_v, rtol=1e-13, atol=1e-14)


def test_mix_zero_and_one_reduce_to_the_single_rules():
    """beta = 0 is the sampling rule alone, beta = 1 is VDN alone (the paper's remark under Eq. 4)."""
    x, dy, gamma, beta, xv, dyv = small(42)
    N, C, H, W = x.shape
    for name, sp in rules(N, C, H, W, 42).items():
        f0 = O.forward_mixed(x, xv, gamma, beta, EPS, 0.0, sp)
        b0 = O.backward_mixed(x, xv, dy, None, gamma, f0, EPS, 0.0, sp)
        f = O.forward(x, gamma, beta, EPS, sp)
        b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
        np.testing.assert_allclose(f0.y, f.y, rtol=1e-13, atol=1e-13, err_msg=name)
        np.testing.assert_allclose(b0.dx, b.dx, rtol=1e-12, atol=1e-13, err_msg=name)
        np.testing.assert_allclose(b0.dgamma, b.dgamma, rtol=1e-12, err_msg=name)
        f1 = O.forward_mixed(x, xv, gamma, beta, EPS, 1.0, sp)
        b1 = O.backward_mixed(x, xv, dy, dyv, gamma, f1, EPS, 1.0, sp)
        fv = O.forward(x, gamma, beta, EPS, O.Sampling.virtual(xv.shape[0]), xv=xv)
        bv = O.backward(x, dy, gamma, fv.mean, fv.var, EPS, O.Sampling.virtual(xv.shape[0]), xv=xv, dyv=dyv)
        np.testing.assert_allclose(f1.y, fv.y, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(f1.yv, fv.yv, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(b1.dx, bv.dx, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(b1.dxv, bv.dxv, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(b1.dbeta, bv.dbeta, rtol=1e-12)


def autograd_mixed(x, xv, dy, dyv, gamma, beta, eps, mix, mask):
    """Eq. 1 + Eq. 3 + Eq. 4 written with torch ops; the gradient comes from autograd."""
    t = lambda a: torch.tensor(a, dtype=torch.float64)
    xt, xvt = t(x).requires_grad_(), t(xv).requires_grad_()
    gt, bt = t(gamma).requires_grad_(), t(beta).requires_grad_()
    mt = t(mask)
    sh = (1, -1, 1, 1)
    s = mt.sum(dim=(0, 2, 3))
    mean_s = (xt * mt).sum(dim=(0, 2, 3)) / s
    var_s = (((xt - mean_s.view(sh)) ** 2) * mt).sum(dim=(0, 2, 3)) / s
    mean_v, var_v = xvt.mean(dim=(0, 2, 3)), xvt.var(dim=(0, 2, 3), unbiased=False)
    mean, var = mix * mean_v + (1 - mix) * mean_s, mix * var_v + (1 - mix) * var_s
    norm = lambda a: gt.view(sh) * (a - mean.view(sh)) / torch.sqrt(var.view(sh) + eps) + bt.view(sh)
    loss = (norm(xt) * t(dy)).sum()
    if dyv is not None:
        loss = loss + (norm(xvt) * t(dyv)).sum()
    loss.backward()
    return xt.grad.numpy(), xvt.grad.numpy(), gt.grad.numpy(), bt.grad.numpy()


@pytest.mark.parametrize("with_dyv", [True, False])
def test_mixed_backward_matches_autograd(with_dyv):
    x, dy, gamma, beta, xv, dyv = small(43)
    N, C, H, W = x.shape
    for name, sp in rules(N, C, H, W, 43).items():
        for mix in (0.5, 0.2):
            f = O.forward_mixed(x, xv, gamma, beta, EPS, mix, sp)
            b = O.backward_mixed(x, xv, dy, dyv if with_dyv else None, gamma, f, EPS, mix, sp)
            mask = O.selection_mask(N, C, H, W, sp)
            dx, dxv, dg, db = autograd_mixed(x, xv, dy, dyv if with_dyv else None, gamma, beta, EPS, mix, mask)
            np.testing.assert_allclose(b.dx, dx, rtol=1e-10, atol=1e-12, err_msg=name)
            np.testing.assert_allclose(b.dxv, dxv, rtol=1e-10, atol=1e-12, err_msg=name)
            np.testing.assert_allclose(b.dgamma, dg, rtol=1e-11, atol=1e-12, err_msg=name)
            np.testing.assert_allclose(b.dbeta, db, rtol=1e-11, atol=1e-12, err_msg=name)


def test_mixed_backward_finite_differences():
    q = 2.0 ** -10
    snap = lambda a: (np.round(a / q) * q).astype(np.float32)
    x, dy, gamma, beta, xv, dyv = (snap(a) for a in small(44))
    N, C, H, W = x.shape
    sp = rules(N, C, H, W, 44)["feature"]
    mix, h = 0.5, np.float32(2.0 ** -7)

    def loss(xa, xva):
        f = O.forward_mixed(xa, xva, gamma, beta, EPS, mix, sp)
        return (f.y * dy).sum() + (f.yv * dyv).sum()

    f = O.forward_mixed(x, xv, gamma, beta, EPS, mix, sp)
    b = O.backward_mixed(x, xv, dy, dyv, gamma, f, EPS, mix, sp)
    rng = np.random.default_rng(1)
    for arr, grad, which in ((x, b.dx, 0), (xv, b.dxv, 1)):
        for p in rng.choice(arr.size, 10, replace=False):
            idx = np.unravel_index(p, arr.shape)
            est = []
            for m in (1, 2):
                ap, am = arr.copy(), arr.copy()
                ap[idx] += m * h
                am[idx] -= m * h
                lp = loss(ap, xv) if which == 0 else loss(x, ap)
                lm = loss(am, xv) if which == 0 else loss(x, am)
                est.append((lp - lm) / (2.0 * m * float(h)))
            fd = (4.0 * est[0] - est[1]) / 3.0
            assert abs(fd - grad[idx]) < 2e-6 * max(1.0, abs(grad[idx])), (which, idx, fd, grad[idx])


# --------------------------------------------------------------------------- Appendix D
def test_moving_average_recursion_and_closed_form():
    rng = np.random.default_rng(2)
    alpha, T, C = 0.7, 12, 5
    X = rng.normal(size=(T, C))
    ma = None
    for it in range(T):
        ma = O.moving_average(X[it], ma, alpha, first_iteration=(it == 0))
    # unrolled Eq. 8: X_ma,T = (1-a)^(T-1) X_1 + sum_{t>=2} a (1-a)^(T-t) X_t
    w = np.array([(1 - alpha) ** (T - 1)] + [alpha * (1 - alpha) ** (T - t) for t in range(2, T + 1)])
    np.testing.assert_allclose(ma, (w[:, None] * X).sum(axis=0), rtol=1e-13)
    assert abs(w.sum() - 1.0) < 1e-14
    # a constant statistic stays put; the first iteration copies
    c = np.full(C, 3.5)
    assert np.array_equal(O.moving_average(c, None, alpha, True), c)
    np.testing.assert_allclose(O.moving_average(c, c, alpha, False), c, rtol=1e-15)


def test_moving_average_variance_follows_eq9():
    """Eq. 9: for iid estimates, Var[X_ma] ~ alpha/(2-alpha) Var[X] - which also fixes that alpha weights
    the NEW value (with the roles swapped the ratio would be (1-alpha)/(1+alpha))."""
    rng = np.random.default_rng(3)
    alpha, T, C = 0.7, 60, 40000
    X = rng.normal(size=(T, C))
    ma = None
    for it in range(T):
        ma = O.moving_average(X[it], ma, alpha, first_iteration=(it == 0))
    ratio = ma.var() / X.var()
    assert abs(ratio - alpha / (2 - alpha)) < 0.02
    assert abs(ratio - (1 - alpha) / (1 + alpha)) > 0.3


def test_inference_forward_is_library_eval_batch_norm():
    x, dy, gamma, beta, xv, dyv = small(45)
    C = x.shape[1]
    rng = np.random.default_rng(4)
    E_ma, Var_ma = rng.normal(size=C), rng.uniform(0.5, 2.0, size=C)
    y = O.inference_forward(x, gamma, beta, EPS, E_ma, Var_ma)
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    want = torch.nn.functional.batch_norm(t(x), t(E_ma), t(Var_ma), t(gamma), t(beta), training=False, eps=EPS)
    np.testing.assert_allclose(y, want.numpy(), rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------- BN + residual + ReLU
@pytest.mark.parametrize("with_residual", [True, False])
def test_relu_composition_matches_autograd(with_residual):
    x, dy, gamma, beta, xv, dyv = small(46)
    N, C, H, W = x.shape
    res = I.upstream_gradient(x.shape, 46, I.TAG_XV) if with_residual else None
    for name, sp in list(rules(N, C, H, W, 46).items()) + [("full", O.Sampling.full())]:
        f = O.forward_relu(x, res, gamma, beta, EPS, sp)
        b, dres = O.backward_relu(x, dy, gamma, f, EPS, sp)
        t = lambda a: torch.tensor(a, dtype=torch.float64)
        xt, gt, bt = t(x).requires_grad_(), t(gamma).requires_grad_(), t(beta).requires_grad_()
        rt = t(res).requires_grad_() if with_residual else None
        mt = t(O.selection_mask(N, C, H, W, sp))
        sh = (1, -1, 1, 1)
        s = mt.sum(dim=(0, 2, 3))
        mean = (xt * mt).sum(dim=(0, 2, 3)) / s
        var = (((xt - mean.view(sh)) ** 2) * mt).sum(dim=(0, 2, 3)) / s
        z = gt.view(sh) * (xt - mean.view(sh)) / torch.sqrt(var.view(sh) + EPS) + bt.view(sh)
        if with_residual:
            z = z + rt
        y = torch.relu(z)
        (y * t(dy)).sum().backward()
        np.testing.assert_allclose(f.y, y.detach().numpy(), rtol=1e-12, atol=1e-13, err_msg=name)
        np.testing.assert_allclose(b.dx, xt.grad.numpy(), rtol=1e-10, atol=1e-12, err_msg=name)
        np.testing.assert_allclose(b.dgamma, gt.grad.numpy(), rtol=1e-11, atol=1e-12, err_msg=name)
        np.testing.assert_allclose(b.dbeta, bt.grad.numpy(), rtol=1e-11, atol=1e-12, err_msg=name)
        if with_residual:
            np.testing.assert_allclose(dres, rt.grad.numpy(), rtol=0, atol=0, err_msg=name)
