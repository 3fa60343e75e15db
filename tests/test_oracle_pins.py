"""Pins for the CPU oracle: each checks it against something the paper or the mathematics fixes,
not against itself."""
import os

import numpy as np
import pytest
import torch

import bns_inputs as I
import oracle as O

EPS = 1e-5


def small(seed, N=6, C=5, H=7, W=9):
    x = I.tiny_activations(N, C, H, W, seed)
    dy = I.upstream_gradient(x.shape, seed)
    gamma, beta = I.affine_parameters(C, seed)
    return x, dy, gamma, beta


def rules(N, C, H, W, seed):
    """One Sampling of every kind that fits the shape (VIRTUAL separately: it needs xv)."""
    return {
        "batch_paper": O.Sampling.batch(I.batch_sample_indices(N, 2, seed, contiguous=True)),
        "batch_any": O.Sampling.batch(np.array([N - 1, 0, 2], dtype=np.int32)),
        "feature_shared": O.Sampling.feature(3, 4, I.patch_offsets(N, C, H, W, 3, 4, I.OFFSETS_SHARED, seed)),
        "feature_sample": O.Sampling.feature(2, 2, I.patch_offsets(N, C, H, W, 2, 2, I.OFFSETS_PER_SAMPLE, seed),
                                             O.OFFSETS_PER_SAMPLE),
        "feature_map": O.Sampling.feature(1, 3, I.patch_offsets(N, C, H, W, 1, 3, I.OFFSETS_PER_MAP, seed),
                                          O.OFFSETS_PER_MAP),
        "full": O.Sampling.full(),
    }


def numpy_mask(N, C, H, W, sp):
    """The paper's slices (Algorithms 1-2) written with numpy indexing."""
    m = np.zeros((N, C, H, W), dtype=np.uint8)
    if sp.rule == O.RULE_FULL:
        m[:] = 1
    elif sp.rule == O.RULE_BATCH:
        m[sp.sample_idx] = 1
    elif sp.rule == O.RULE_FEATURE:
        for n in range(N):
            for c in range(C):
                e = {O.OFFSETS_SHARED: 0, O.OFFSETS_PER_SAMPLE: n, O.OFFSETS_PER_MAP: n * C + c}[sp.offset_mode]
                oh, ow = sp.offsets[e]
                m[n, c, oh:oh + sp.ph, ow:ow + sp.pw] = 1
    return m


# --------------------------------------------------------------------------- the paper's one worked number
def test_adder_tree_worked_example():
    path = os.path.join(os.path.dirname(__file__), "golden", "adder_tree_speedup.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    for N, H, W, denom, speedup, visited in rows:
        N, H, W, denom = int(N), int(H), int(W), int(denom)
        sp = O.Sampling.batch(np.arange(N // denom, dtype=np.int32))
        m = N * H * W
        assert O.sample_count(N, H, W, O.Sampling.full()) == m
        assert O.sample_count(N, H, W, sp) == m // denom
        ratio = O.adder_tree_depth_ratio(N, H, W, sp)
        assert round((ratio - 1.0) * 100.0, 1) == float(speedup)
        assert round(100.0 * O.sample_count(N, H, W, sp) / m, 1) == float(visited)


def test_sample_counts():
    N, C, H, W = 6, 5, 7, 9
    for name, sp in rules(N, C, H, W, 3).items():
        per_channel = numpy_mask(N, C, H, W, sp).sum(axis=(0, 2, 3))
        assert (per_channel == O.sample_count(N, H, W, sp)).all(), name
    assert O.sample_count(N, H, W, O.Sampling.virtual(2)) == 2 * H * W


# --------------------------------------------------------------------------- selection
def test_selection_mask_matches_paper_slices():
    N, C, H, W = 6, 5, 7, 9
    for name, sp in rules(N, C, H, W, 7).items():
        assert np.array_equal(O.selection_mask(N, C, H, W, sp), numpy_mask(N, C, H, W, sp)), name
    assert O.selection_mask(N, C, H, W, O.Sampling.virtual(2)).sum() == 0


def test_selection_sentinel():
    """x is 1 on S and 0 elsewhere -> mean 1, var 0; x is 1 off S and 0 on S -> mean 0."""
    N, C, H, W = 6, 5, 7, 9
    gamma, beta = np.ones(C, np.float32), np.zeros(C, np.float32)
    for name, sp in rules(N, C, H, W, 11).items():
        on = numpy_mask(N, C, H, W, sp).astype(np.float32)
        f = O.forward(on, gamma, beta, EPS, sp)
        assert np.array_equal(f.mean, np.ones(C)) and np.array_equal(f.var, np.zeros(C)), name
        f = O.forward(1.0 - on, gamma, beta, EPS, sp)
        assert np.array_equal(f.mean, np.zeros(C)) and np.array_equal(f.var, np.zeros(C)), name


# --------------------------------------------------------------------------- statistics
def test_statistics_match_numpy_on_slices(tiny_case):
    t = tiny_case
    x = t["x"].astype(np.float64)
    N, C, H, W = x.shape
    # Algorithm 1: B[idx] ; Eq. 3 is numpy's mean / biased var over dims (0,2,3)
    f = O.forward(t["x"], t["gamma"], t["beta"], EPS, O.Sampling.batch(t["idx"]))
    xs = x[t["idx"]]
    np.testing.assert_allclose(f.mean, xs.mean(axis=(0, 2, 3)), rtol=0, atol=1e-14)
    np.testing.assert_allclose(f.var, xs.var(axis=(0, 2, 3), ddof=0), rtol=1e-13)
    np.testing.assert_allclose(f.invstd, 1.0 / np.sqrt(xs.var(axis=(0, 2, 3)) + EPS), rtol=1e-13)
    # Algorithm 2: B[:, :, oh:oh+ph, ow:ow+pw]
    off = I.patch_offsets(N, C, H, W, 3, 2, I.OFFSETS_SHARED, 5)
    f = O.forward(t["x"], t["gamma"], t["beta"], EPS, O.Sampling.feature(3, 2, off))
    xs = x[:, :, off[0, 0]:off[0, 0] + 3, off[0, 1]:off[0, 1] + 2]
    np.testing.assert_allclose(f.mean, xs.mean(axis=(0, 2, 3)), rtol=0, atol=1e-14)
    np.testing.assert_allclose(f.var, xs.var(axis=(0, 2, 3)), rtol=1e-13)
    # Algorithm 3: virtual rows only
    xv = I.virtual_samples(2, C, H, W, 5)
    f = O.forward(t["x"], t["gamma"], t["beta"], EPS, O.Sampling.virtual(2), xv=xv)
    np.testing.assert_allclose(f.mean, xv.astype(np.float64).mean(axis=(0, 2, 3)), rtol=0, atol=1e-14)
    np.testing.assert_allclose(f.var, xv.astype(np.float64).var(axis=(0, 2, 3)), rtol=1e-13)
    # biased, not Bessel-corrected
    assert not np.allclose(f.var, xv.astype(np.float64).var(axis=(0, 2, 3), ddof=1), rtol=1e-6)


def test_forward_is_eq1_with_those_statistics(tiny_case):
    t = tiny_case
    f = O.forward(t["x"], t["gamma"], t["beta"], EPS, O.Sampling.batch(t["idx"]))
    x = t["x"].astype(np.float64)
    g, b = t["gamma"].astype(np.float64), t["beta"].astype(np.float64)
    sh = (1, -1, 1, 1)
    y = g.reshape(sh) * (x - f.mean.reshape(sh)) / np.sqrt(f.var.reshape(sh) + EPS) + b.reshape(sh)
    np.testing.assert_allclose(f.y, y, rtol=1e-13, atol=1e-14)


def test_sampled_set_is_standardised():
    x, dy, gamma, beta = small(21)
    N, C, H, W = x.shape
    one, zero = np.ones(C, np.float32), np.zeros(C, np.float32)
    for name, sp in rules(N, C, H, W, 21).items():
        f = O.forward(x, one, zero, EPS, sp)
        m = numpy_mask(N, C, H, W, sp).astype(bool)
        s = O.sample_count(N, H, W, sp)
        for c in range(C):
            xh = f.y[:, c][m[:, c]]
            assert xh.size == s
            assert abs(xh.sum()) < 1e-10 * s, name
            np.testing.assert_allclose((xh ** 2).sum() / s, f.var[c] / (f.var[c] + EPS), rtol=1e-12, err_msg=name)


def test_affine_equivariance_and_constant_input():
    x, dy, gamma, beta = small(22)
    x = (np.round(x * 1024.0) / 1024.0).astype(np.float32)   # on a 2^-10 grid, so 2x+4 is exact in fp32
    N, C, H, W = x.shape
    for name, sp in rules(N, C, H, W, 22).items():
        f1 = O.forward(x, gamma, beta, EPS, sp)
        f2 = O.forward(np.float32(2.0) * x + np.float32(4.0), gamma, beta, EPS, sp)   # exact in fp32
        np.testing.assert_allclose(f2.mean, 2.0 * f1.mean + 4.0, rtol=1e-12, err_msg=name)
        np.testing.assert_allclose(f2.var, 4.0 * f1.var, rtol=1e-12, err_msg=name)
        fc = O.forward(np.full_like(x, 3.25), gamma, beta, EPS, sp)
        assert np.array_equal(fc.var, np.zeros(C)) and np.array_equal(fc.mean, np.full(C, 3.25))
        np.testing.assert_allclose(fc.invstd, EPS ** -0.5, rtol=1e-15)
        np.testing.assert_allclose(fc.y, np.broadcast_to(beta.astype(np.float64).reshape(1, -1, 1, 1), x.shape))


# --------------------------------------------------------------------------- ratio 1 and the library operator
def torch_batch_norm(x, dy, gamma, beta, eps):
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    gt = torch.tensor(gamma, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(beta, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.batch_norm(xt, None, None, gt, bt, training=True, eps=eps)
    y.backward(torch.tensor(dy, dtype=torch.float64))
    return y.detach().numpy(), xt.grad.numpy(), gt.grad.numpy(), bt.grad.numpy()


def test_ratio_one_is_full_bn_and_library_batch_norm():
    x, dy, gamma, beta = small(23)
    N, C, H, W = x.shape
    y_t, dx_t, dg_t, db_t = torch_batch_norm(x, dy, gamma, beta, EPS)
    full = O.forward(x, gamma, beta, EPS, O.Sampling.full())
    fullb = O.backward(x, dy, gamma, full.mean, full.var, EPS, O.Sampling.full())
    np.testing.assert_allclose(full.y, y_t, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(fullb.dx, dx_t, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(fullb.dgamma, dg_t, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(fullb.dbeta, db_t, rtol=1e-12, atol=1e-12)
    ratio_one = [O.Sampling.batch(np.arange(N, dtype=np.int32)),
                 O.Sampling.feature(H, W, np.zeros((1, 2), np.int32)),
                 O.Sampling.feature(H, W, np.zeros((N * C, 2), np.int32), O.OFFSETS_PER_MAP)]
    for sp in ratio_one:
        f = O.forward(x, gamma, beta, EPS, sp)
        b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
        for got, want in ((f.y, full.y), (f.mean, full.mean), (f.var, full.var), (b.dx, fullb.dx),
                          (b.dgamma, fullb.dgamma), (b.dbeta, fullb.dbeta)):
            assert np.array_equal(got, want)


def test_full_bn_gradient_identities():
    x, dy, gamma, beta = small(24)
    one, zero = np.ones_like(gamma), np.zeros_like(beta)
    f = O.forward(x, one, zero, EPS, O.Sampling.full())
    b = O.backward(x, dy, gamma, f.mean, f.var, EPS, O.Sampling.full())
    assert np.abs(b.dx.sum(axis=(0, 2, 3))).max() < 1e-12
    # sum(dx * xhat) = gamma*invstd*dgamma * eps/(var+eps): zero but for eps
    want = gamma * f.invstd * b.dgamma * EPS / (f.var + EPS)
    np.testing.assert_allclose((b.dx * f.y).sum(axis=(0, 2, 3)), want, rtol=1e-7, atol=1e-12)
    np.testing.assert_allclose(b.dbeta, dy.astype(np.float64).sum(axis=(0, 2, 3)), rtol=1e-13)
    np.testing.assert_allclose(b.dgamma, (dy.astype(np.float64) * f.y).sum(axis=(0, 2, 3)), rtol=1e-12)


# --------------------------------------------------------------------------- backward: autograd and finite differences
def autograd_reference(x, dy, gamma, beta, eps, mask, xv=None, dyv=None):
    """The forward definition (Eq. 1 + Eq. 3) written with torch ops on a 0/1 mask; its gradient
    comes from autograd, not from Eq. 5/6."""
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    gt = torch.tensor(gamma, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(beta, dtype=torch.float64, requires_grad=True)
    sh = (1, -1, 1, 1)
    if xv is None:
        mt = torch.tensor(mask, dtype=torch.float64)
        s = mt.sum(dim=(0, 2, 3))
        mean = (xt * mt).sum(dim=(0, 2, 3)) / s
        var = (((xt - mean.view(sh)) ** 2) * mt).sum(dim=(0, 2, 3)) / s
        xvt = None
    else:
        xvt = torch.tensor(xv, dtype=torch.float64, requires_grad=True)
        mean = xvt.mean(dim=(0, 2, 3))
        var = xvt.var(dim=(0, 2, 3), unbiased=False)
    norm = lambda t: gt.view(sh) * (t - mean.view(sh)) / torch.sqrt(var.view(sh) + eps) + bt.view(sh)
    loss = (norm(xt) * torch.tensor(dy, dtype=torch.float64)).sum()
    if xvt is not None and dyv is not None:
        loss = loss + (norm(xvt) * torch.tensor(dyv, dtype=torch.float64)).sum()
    loss.backward()
    return (xt.grad.numpy(), gt.grad.numpy(), bt.grad.numpy(),
            None if xvt is None else (xvt.grad.numpy() if xvt.grad is not None else np.zeros_like(xv)))


def test_backward_matches_autograd_of_the_definition():
    x, dy, gamma, beta = small(25)
    N, C, H, W = x.shape
    for name, sp in rules(N, C, H, W, 25).items():
        f = O.forward(x, gamma, beta, EPS, sp)
        b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
        dx, dg, db, _ = autograd_reference(x, dy, gamma, beta, EPS, numpy_mask(N, C, H, W, sp))
        np.testing.assert_allclose(b.dx, dx, rtol=1e-10, atol=1e-12, err_msg=name)
        np.testing.assert_allclose(b.dgamma, dg, rtol=1e-11, atol=1e-12, err_msg=name)
        np.testing.assert_allclose(b.dbeta, db, rtol=1e-11, atol=1e-12, err_msg=name)


@pytest.mark.parametrize("with_dyv", [True, False])
def test_virtual_backward_matches_autograd(with_dyv):
    x, dy, gamma, beta = small(26)
    N, C, H, W = x.shape
    xv = I.virtual_samples(2, C, H, W, 26)
    dyv = I.upstream_gradient(xv.shape, 26, I.TAG_DYV) if with_dyv else None
    sp = O.Sampling.virtual(2)
    f = O.forward(x, gamma, beta, EPS, sp, xv=xv)
    b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp, xv=xv, dyv=dyv)
    dx, dg, db, dxv = autograd_reference(x, dy, gamma, beta, EPS, None, xv=xv, dyv=dyv)
    np.testing.assert_allclose(b.dx, dx, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(b.dxv, dxv, rtol=1e-10, atol=1e-12)
    if with_dyv:
        np.testing.assert_allclose(b.dgamma, dg, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(b.dbeta, db, rtol=1e-11, atol=1e-12)


def loss_of(x, dy, gamma, beta, sp, xv=None, dyv=None):
    """Finite differences perturb float32 inputs, so perturb in float64 and feed the oracle values
    that are exactly representable: work on a grid of 2^-12."""
    f = O.forward(x, gamma, beta, EPS, sp, xv=xv)
    l = (f.y * dy.astype(np.float64)).sum()
    if xv is not None and dyv is not None:
        l += (f.yv * dyv.astype(np.float64)).sum()
    return l


def test_backward_matches_finite_differences(tiny_case):
    """Central differences of L = sum(dy * y) on config 1 (inputs snapped to a 2^-10 grid so that
    x +- h stays exact in float32)."""
    t = tiny_case
    q = 2.0 ** -10
    snap = lambda a: (np.round(a / q) * q).astype(np.float32)
    x, dy, gamma, beta = snap(t["x"]), snap(t["dy"]), snap(t["gamma"]), snap(t["beta"])
    N, C, H, W = x.shape
    h = np.float32(2.0 ** -7)
    cases = {"batch": (O.Sampling.batch(t["idx"]), None, None),
             "feature": (O.Sampling.feature(3, 3, I.patch_offsets(N, C, H, W, 3, 3, I.OFFSETS_PER_SAMPLE, 9),
                                            O.OFFSETS_PER_SAMPLE), None, None),
             "virtual": (O.Sampling.virtual(2), snap(I.virtual_samples(2, C, H, W, 9)),
                         snap(I.upstream_gradient((2, C, H, W), 9, I.TAG_DYV)))}
    rng = np.random.default_rng(0)
    for name, (sp, xv, dyv) in cases.items():
        f = O.forward(x, gamma, beta, EPS, sp, xv=xv)
        b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp, xv=xv, dyv=dyv)
        mask = O.selection_mask(N, C, H, W, sp)
        # probe sampled and non-sampled positions alike
        flat_on, flat_off = np.flatnonzero(mask), np.flatnonzero(mask == 0)
        probes = list(rng.choice(flat_off, 12, replace=False))
        if flat_on.size:
            probes += list(rng.choice(flat_on, 12, replace=False))
        for p in probes:
            idx = np.unravel_index(p, x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            fd = (loss_of(xp, dy, gamma, beta, sp, xv, dyv) - loss_of(xm, dy, gamma, beta, sp, xv, dyv)) / (2.0 * float(h))
            # Richardson step to cancel the h^2 term
            xp2, xm2 = x.copy(), x.copy()
            xp2[idx] += 2 * h
            xm2[idx] -= 2 * h
            fd2 = (loss_of(xp2, dy, gamma, beta, sp, xv, dyv) - loss_of(xm2, dy, gamma, beta, sp, xv, dyv)) / (4.0 * float(h))
            est = (4.0 * fd - fd2) / 3.0
            assert abs(est - b.dx[idx]) < 2e-6 * max(1.0, abs(b.dx[idx])), (name, idx, est, b.dx[idx])
        if xv is not None:
            for p in rng.choice(xv.size, 12, replace=False):
                idx = np.unravel_index(p, xv.shape)
                vals = []
                for mult in (1, 2):
                    vp, vm = xv.copy(), xv.copy()
                    vp[idx] += mult * h
                    vm[idx] -= mult * h
                    vals.append((loss_of(x, dy, gamma, beta, sp, vp, dyv) - loss_of(x, dy, gamma, beta, sp, vm, dyv))
                                / (2.0 * mult * float(h)))
                est = (4.0 * vals[0] - vals[1]) / 3.0
                assert abs(est - b.dxv[idx]) < 2e-6 * max(1.0, abs(b.dxv[idx])), (name, idx)
        # gamma and beta: L is linear in both, so the difference quotient is exact up to rounding
        for c in range(0, C, 5):
            for arr, grad in ((gamma, b.dgamma), (beta, b.dbeta)):
                ap, am = arr.copy(), arr.copy()
                ap[c] += h
                am[c] -= h
                if arr is gamma:
                    lp, lm = loss_of(x, dy, ap, beta, sp, xv, dyv), loss_of(x, dy, am, beta, sp, xv, dyv)
                else:
                    lp, lm = loss_of(x, dy, gamma, ap, sp, xv, dyv), loss_of(x, dy, gamma, am, sp, xv, dyv)
                assert abs((lp - lm) / (2.0 * float(h)) - grad[c]) < 1e-9 * max(1.0, abs(grad[c])), name


def test_sampled_gradient_identities():
    """Off S the gradient is exactly gamma*invstd*dy; on S the correction sums to a known value."""
    x, dy, gamma, beta = small(27)
    N, C, H, W = x.shape
    for name, sp in rules(N, C, H, W, 27).items():
        f = O.forward(x, gamma, beta, EPS, sp)
        b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
        m = numpy_mask(N, C, H, W, sp).astype(bool)
        g = gamma.astype(np.float64)
        for c in range(C):
            base = g[c] * dy[:, c].astype(np.float64) / np.sqrt(f.var[c] + EPS)
            assert np.array_equal(b.dx[:, c][~m[:, c]], base[~m[:, c]]), name
            lhs = b.dx[:, c][m[:, c]].sum()
            rhs = g[c] * f.invstd[c] * (dy[:, c][m[:, c]].astype(np.float64).sum() - b.dbeta[c])
            np.testing.assert_allclose(lhs, rhs, rtol=1e-10, atol=1e-10, err_msg=name)


# --------------------------------------------------------------------------- equivalences between the rules
def test_rule_equivalences():
    x, dy, gamma, beta = small(28)
    N, C, H, W = x.shape
    run = lambda sp, **kw: (O.forward(x, gamma, beta, EPS, sp, **kw))
    # Naive Sampling is Batch Sampling with begin = 0 (Algorithm 1)
    ns = run(O.Sampling.batch(np.arange(3, dtype=np.int32)))
    np.testing.assert_allclose(ns.mean, x[:3].astype(np.float64).mean(axis=(0, 2, 3)), atol=1e-14)
    # the order of the sample list does not matter (up to summation order)
    a = run(O.Sampling.batch(np.array([4, 1, 3], np.int32)))
    b = run(O.Sampling.batch(np.array([1, 3, 4], np.int32)))
    np.testing.assert_allclose(a.y, b.y, rtol=1e-13, atol=1e-13)
    # per-map offsets that are all equal reproduce the shared location exactly
    off = np.array([[2, 3]], np.int32)
    shared = O.Sampling.feature(3, 4, off)
    per_map = O.Sampling.feature(3, 4, np.repeat(off, N * C, axis=0), O.OFFSETS_PER_MAP)
    per_sample = O.Sampling.feature(3, 4, np.repeat(off, N, axis=0), O.OFFSETS_PER_SAMPLE)
    fs = run(shared)
    bs = O.backward(x, dy, gamma, fs.mean, fs.var, EPS, shared)
    for sp in (per_map, per_sample):
        f = run(sp)
        bb = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
        assert np.array_equal(f.y, fs.y) and np.array_equal(bb.dx, bs.dx) and np.array_equal(bb.dgamma, bs.dgamma)


def test_virtual_equals_batch_on_concatenated_batch():
    """Algorithm 3 puts the virtual samples in front of the batch and takes rows 0..nv-1."""
    x, dy, gamma, beta = small(29)
    N, C, H, W = x.shape
    nv = 2
    xv = I.virtual_samples(nv, C, H, W, 29)
    dyv = I.upstream_gradient(xv.shape, 29, I.TAG_DYV)
    fv = O.forward(x, gamma, beta, EPS, O.Sampling.virtual(nv), xv=xv)
    bv = O.backward(x, dy, gamma, fv.mean, fv.var, EPS, O.Sampling.virtual(nv), xv=xv, dyv=dyv)
    xc, dyc = np.concatenate([xv, x]), np.concatenate([dyv, dy])
    sp = O.Sampling.batch(np.arange(nv, dtype=np.int32))
    fc = O.forward(xc, gamma, beta, EPS, sp)
    bc = O.backward(xc, dyc, gamma, fc.mean, fc.var, EPS, sp)
    assert np.array_equal(fv.mean, fc.mean) and np.array_equal(fv.var, fc.var)
    assert np.array_equal(fv.yv, fc.y[:nv]) and np.array_equal(fv.y, fc.y[nv:])
    np.testing.assert_allclose(bv.dgamma, bc.dgamma, rtol=1e-13)
    np.testing.assert_allclose(bv.dbeta, bc.dbeta, rtol=1e-13)
    np.testing.assert_allclose(bv.dxv, bc.dx[:nv], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(bv.dx, bc.dx[nv:], rtol=1e-12, atol=1e-14)


def test_channel_subset_is_the_same_computation():
    x, dy, gamma, beta = small(30)
    N, C, H, W = x.shape
    sp = O.Sampling.feature(2, 5, I.patch_offsets(N, C, H, W, 2, 5, I.OFFSETS_PER_MAP, 30), O.OFFSETS_PER_MAP)
    f = O.forward(x, gamma, beta, EPS, sp)
    b = O.backward(x, dy, gamma, f.mean, f.var, EPS, sp)
    ch = np.array([3, 0], np.int32)
    fs = O.forward(x, gamma, beta, EPS, sp, channels=ch)
    bs = O.backward(x, dy, gamma, fs.mean, fs.var, EPS, sp, channels=ch)
    assert np.array_equal(fs.y, f.y[:, ch]) and np.array_equal(fs.mean, f.mean[ch])
    assert np.array_equal(bs.dx, b.dx[:, ch]) and np.array_equal(bs.dgamma, b.dgamma[ch])
