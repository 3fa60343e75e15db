"""GPU parity for the rows beyond the basic path: VDN combined with a sampling rule (Eq. 4), the moving
average of the statistics (Eq. 8) and the validation-time forward (Appendix D)."""
import numpy as np
import pytest

import bns_inputs as I
import oracle as O
from helpers import _to_device, _to_host, close_bf16, close_f32, gpu_sampling, make_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=3, contiguous=False)), ("batch", dict(k=8)), ("feature", dict(ph=3, pw=3, offset_mode=0)),
    ("feature", dict(ph=2, pw=5, offset_mode=2)),
])
@pytest.mark.parametrize("dtype,dims", [("f32", (40, 24, 20, 20)), ("bf16", (32, 48, 14, 14)), ("f32", (9, 5, 7, 7))])
@pytest.mark.parametrize("mix,with_dyv", [(0.5, True), (0.25, False)])
def test_mixed_statistics_forward_backward(rule, kw, dtype, dims, mix, with_dyv):
    _check_mixed(rule, kw, dtype, dims, mix, with_dyv)


def test_mixed_statistics_at_benchmark_size():
    """The shape and rule that bench.py times as `fs_vdn`: 256x64x56x56 fp32, 8x8 patch, two virtual samples."""
    _check_mixed("feature", dict(ph=8, pw=8, offset_mode=0), "f32", (256, 64, 56, 56), 0.5, False)


def _check_mixed(rule, kw, dtype, dims, mix, with_dyv):
    import torch
    from paper_1810_10962_b200 import bns
    case = make_case(*dims, rule, seed=93, dtype=dtype, **kw)
    N, C, H, W = dims
    xv_np = I.virtual_samples(2, C, H, W, 93)
    dyv_np = I.upstream_gradient(xv_np.shape, 93, I.TAG_DYV) if with_dyv else None
    x, dy = _to_device(case.x, dtype), _to_device(case.dy, dtype)
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    xv = torch.from_numpy(xv_np).cuda()
    dyv = torch.from_numpy(dyv_np).cuda() if with_dyv else None
    sp = gpu_sampling(case).with_virtual(xv, yv=torch.empty_like(xv), dyv=dyv, dxv=torch.empty_like(xv))
    y, mean, invstd, mean_s, mean_v = bns.forward_mixed(x, gamma, beta, case.eps, mix, sp)
    dx, dgamma, dbeta = bns.backward_mixed(x, dy, gamma, mean, invstd, mean_s, mean_v, mix, sp)
    torch.cuda.synchronize()
    osp = case.oracle_sampling()
    f = O.forward_mixed(case.x, xv_np, case.gamma, case.beta, case.eps, mix, osp)
    b = O.backward_mixed(case.x, xv_np, case.dy, dyv_np, case.gamma, f, case.eps, mix, osp)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    close_f32(mean_s.cpu().numpy(), f.mean_s, "mean_s")
    close_f32(mean_v.cpu().numpy(), f.mean_v, "mean_v")
    tensor_close(_to_host(y), f.y, "y")
    close_f32(sp.yv.cpu().numpy(), f.yv, "yv")
    tensor_close(_to_host(dx), b.dx, "dx")
    close_f32(sp.dxv.cpu().numpy(), b.dxv, "dxv")
    close_f32(dgamma.cpu().numpy(), b.dgamma, "dgamma")
    close_f32(dbeta.cpu().numpy(), b.dbeta, "dbeta")


def test_mixed_rejects_other_rules_and_weights():
    import ctypes
    import torch
    from paper_1810_10962_b200 import bns
    x = torch.zeros(4, 4, 8, 8, device="cuda")
    xv = torch.zeros(2, 4, 8, 8, device="cuda")
    g = torch.ones(4, device="cuda")
    with pytest.raises(bns.BnsError):
        bns.forward_mixed(x, g, g, 1e-5, 0.5, bns.Sampling.virtual(xv))            # needs BATCH or FEATURE
    sp = bns.Sampling.batch(np.array([0, 1], np.int32)).with_virtual(xv)
    with pytest.raises(bns.BnsError):
        bns.forward_mixed(x, g, g, 1e-5, 1.5, sp, workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))


def test_moving_average_and_inference_forward():
    import torch
    from paper_1810_10962_b200 import bns
    N, C, H, W = 32, 24, 10, 10
    gamma_np, beta_np = I.affine_parameters(C, 94)
    gamma, beta = torch.from_numpy(gamma_np).cuda(), torch.from_numpy(beta_np).cuda()
    mean_ma = torch.zeros(C, device="cuda")
    var_ma = torch.zeros(C, device="cuda")
    o_mean = o_var = None
    alpha = 0.7
    for it in range(4):                       # four training iterations with Batch Sampling, different batches
        x_np = I.correlated_activations(N, C, H, W, 940 + it)
        idx = I.batch_sample_indices(N, 4, 940 + it, contiguous=True)
        x = torch.from_numpy(x_np).cuda()
        _, mean, invstd = bns.forward(x, gamma, beta, 1e-5, bns.Sampling.batch(idx))
        bns.update_moving_average(mean, invstd, 1e-5, alpha, it == 0, mean_ma, var_ma)
        f = O.forward(x_np, gamma_np, beta_np, 1e-5, O.Sampling.batch(idx), want_y=False)
        o_mean = O.moving_average(f.mean, o_mean, alpha, it == 0)
        o_var = O.moving_average(f.var, o_var, alpha, it == 0)
    torch.cuda.synchronize()
    close_f32(mean_ma.cpu().numpy(), o_mean, "mean_ma")
    close_f32(var_ma.cpu().numpy(), o_var, "var_ma")
    for dtype in ("f32", "bf16"):
        xe_np = I.correlated_activations(N, C, H, W, 949)
        if dtype == "bf16":
            xe_np = I.round_to_bf16(xe_np)
        y = bns.inference_forward(_to_device(xe_np, dtype), gamma, beta, 1e-5, mean_ma, var_ma)
        want = O.inference_forward(xe_np, gamma_np, beta_np, 1e-5, mean_ma.cpu().numpy().astype(np.float64),
                                   var_ma.cpu().numpy().astype(np.float64))
        (close_f32 if dtype == "f32" else close_bf16)(_to_host(y), want, f"inference y {dtype}")


@pytest.mark.parametrize("dims,rule,kw", [
    ((48, 24, 20, 20), "batch", dict(k=24)),                     # large sampled set: partial sums + finalize
    ((48, 24, 20, 20), "feature", dict(ph=2, pw=2)),             # small sampled set: one block per channel
    ((32, 16, 8, 8), "full", dict()),                            # small tensor, full BN: the on-chip kernel
    ((16, 8, 14, 14), "virtual", dict(nv=2, with_dyv=False)),
])
def test_forward_with_the_moving_average_folded_in(dims, rule, kw):
    """bns_forward_training over three iterations against the oracle's forward + Eq. 8, through each way the
    library finishes its statistics."""
    import torch
    from paper_1810_10962_b200 import bns
    C = dims[1]
    alpha = 0.7
    mean_ma, var_ma = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda")
    o_mean = o_var = None
    for it in range(3):
        case = make_case(*dims, rule, seed=970 + it, **kw)
        x = _to_device(case.x, "f32")
        gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
        sp = gpu_sampling(case)
        y, mean, invstd = bns.forward_training(x, gamma, beta, case.eps, sp, alpha, it == 0, mean_ma, var_ma)
        f = O.forward(case.x, case.gamma, case.beta, case.eps, case.oracle_sampling(), xv=case.xv)
        o_mean = O.moving_average(f.mean, o_mean, alpha, it == 0)
        o_var = O.moving_average(f.var, o_var, alpha, it == 0)
        torch.cuda.synchronize()
        close_f32(_to_host(y), f.y, "y")
        close_f32(mean.cpu().numpy(), f.mean, "mean")
        close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
        close_f32(mean_ma.cpu().numpy(), o_mean, f"mean_ma after iteration {it}")
        close_f32(var_ma.cpu().numpy(), o_var, f"var_ma after iteration {it}")


@pytest.mark.parametrize("rule", ["batch", "feature", "full"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("ranks", [2, 3])
def test_statistics_shared_by_several_ranks_equal_one_big_batch(rule, dtype, ranks):
    """Sync-BN with sampling: the batch is split over `ranks` slices, each slice goes through the per-rank
    calls, the exchanges are a stack (all-gather) and a sum (all-reduce) on the one GPU, and the result
    must be the oracle's for the whole batch with the union of the ranks' sampled sets."""
    import torch
    from paper_1810_10962_b200 import bns
    from helpers import quantise
    n_local, C, H, W = 8, 20, 12, 12
    N = n_local * ranks
    x_np = quantise(I.correlated_activations(N, C, H, W, 95), dtype)
    dy_np = quantise(I.upstream_gradient(x_np.shape, 95), dtype)
    gamma_np, beta_np = I.affine_parameters(C, 95)
    gamma, beta = torch.from_numpy(gamma_np).cuda(), torch.from_numpy(beta_np).cuda()
    eps = 1e-5
    local_idx = [np.array([1 + r, 5], np.int32) for r in range(ranks)]          # each rank samples two of its slices
    offsets = np.array([[3, 2]], np.int32)
    if rule == "batch":
        osp = O.Sampling.batch(np.concatenate([idx + r * n_local for r, idx in enumerate(local_idx)]))
        sps = [bns.Sampling.batch(idx) for idx in local_idx]
    elif rule == "feature":
        osp = O.Sampling.feature(4, 5, offsets)
        sps = [bns.Sampling.feature(4, 5, offsets) for _ in range(ranks)]
    else:
        osp = O.Sampling.full()
        sps = [bns.Sampling.full() for _ in range(ranks)]
    xs = [_to_device(x_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    dys = [_to_device(dy_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    gathered = torch.stack([bns.sync_local_moments(xs[r], sps[r], eps) for r in range(ranks)])   # "all-gather"
    mean, invstd, count = bns.sync_merge_moments(gathered, eps)
    ys = [bns.sync_normalize(xs[r], gamma, beta, mean, invstd) for r in range(ranks)]
    partial = [bns.sync_backward_sums(xs[r], dys[r], gamma, mean, invstd) for r in range(ranks)]
    sums = torch.stack([p[1] for p in partial]).sum(dim=0)                                        # "all-reduce"
    dxs = [bns.sync_backward_apply(xs[r], dys[r], gamma, mean, invstd, sps[r], sums, count, partial[r][0])
           for r in range(ranks)]
    torch.cuda.synchronize()
    assert np.array_equal(count.cpu().numpy(), np.full(C, O.sample_count(N, H, W, osp), np.float32))
    f = O.forward(x_np, gamma_np, beta_np, eps, osp)
    b = O.backward(x_np, dy_np, gamma_np, f.mean, f.var, eps, osp)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    tensor_close(np.concatenate([_to_host(t) for t in ys]), f.y, "y")
    tensor_close(np.concatenate([_to_host(t) for t in dxs]), b.dx, "dx")
    close_f32(sums[0].cpu().numpy(), b.dbeta, "dbeta")
    close_f32(sums[1].cpu().numpy(), b.dgamma, "dgamma")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_statistics_from_a_fraction_of_the_ranks(dtype):
    """Micro-BN, variant (2) of Sec. 4.3 (Batch Sampling over GPUs): only some ranks contribute statistics.
    Three ranks, the middle one samples nothing (sampling=None): the result must be the oracle's for the whole
    batch with a sampled set that lies in the first and the last slice only."""
    import torch
    from paper_1810_10962_b200 import bns
    from helpers import quantise
    ranks, n_local, C, H, W = 3, 6, 12, 10, 10
    N = ranks * n_local
    x_np = quantise(I.correlated_activations(N, C, H, W, 99), dtype)
    dy_np = quantise(I.upstream_gradient(x_np.shape, 99), dtype)
    gamma_np, beta_np = I.affine_parameters(C, 99)
    gamma, beta = torch.from_numpy(gamma_np).cuda(), torch.from_numpy(beta_np).cuda()
    eps = 1e-5
    local = [np.array([0, 3], np.int32), None, np.array([2, 4, 5], np.int32)]
    osp = O.Sampling.batch(np.concatenate([idx + r * n_local for r, idx in enumerate(local) if idx is not None]))
    sps = [None if idx is None else bns.Sampling.batch(idx) for idx in local]
    xs = [_to_device(x_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    dys = [_to_device(dy_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    gathered = torch.stack([bns.sync_local_moments(xs[r], sps[r], eps) for r in range(ranks)])
    assert float(gathered[1].abs().max()) == 0.0                      # the silent rank: a count of zero
    mean, invstd, count = bns.sync_merge_moments(gathered, eps)
    ys = [bns.sync_normalize(xs[r], gamma, beta, mean, invstd) for r in range(ranks)]
    partial = [bns.sync_backward_sums(xs[r], dys[r], gamma, mean, invstd) for r in range(ranks)]
    sums = torch.stack([p[1] for p in partial]).sum(dim=0)
    dxs = [bns.sync_backward_apply(xs[r], dys[r], gamma, mean, invstd, sps[r], sums, count, partial[r][0])
           for r in range(ranks)]
    torch.cuda.synchronize()
    f = O.forward(x_np, gamma_np, beta_np, eps, osp)
    b = O.backward(x_np, dy_np, gamma_np, f.mean, f.var, eps, osp)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    tensor_close(np.concatenate([_to_host(t) for t in ys]), f.y, "y")
    tensor_close(np.concatenate([_to_host(t) for t in dxs]), b.dx, "dx")
    close_f32(sums[0].cpu().numpy(), b.dbeta, "dbeta")
    close_f32(sums[1].cpu().numpy(), b.dgamma, "dgamma")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("with_dyv", [True, False])
def test_virtual_samples_fed_to_one_rank(dtype, with_dyv):
    """Micro-BN, variant (3) of Sec. 4.3: the virtual samples go to one rank, the others contribute nothing.
    The result must be the oracle's VIRTUAL rule on the whole batch, dxv included."""
    import torch
    from paper_1810_10962_b200 import bns
    from helpers import quantise
    ranks, n_local, C, H, W = 2, 7, 10, 12, 12
    N = ranks * n_local
    x_np = quantise(I.correlated_activations(N, C, H, W, 100), dtype)
    dy_np = quantise(I.upstream_gradient(x_np.shape, 100), dtype)
    xv_np = I.virtual_samples(2, C, H, W, 100)
    dyv_np = I.upstream_gradient(xv_np.shape, 100, I.TAG_DYV) if with_dyv else None
    gamma_np, beta_np = I.affine_parameters(C, 100)
    gamma, beta = torch.from_numpy(gamma_np).cuda(), torch.from_numpy(beta_np).cuda()
    eps = 1e-5
    xv = torch.from_numpy(xv_np).cuda()
    dyv = torch.from_numpy(dyv_np).cuda() if with_dyv else None
    sps = [bns.Sampling.virtual(xv, yv=torch.empty_like(xv), dyv=dyv, dxv=torch.empty_like(xv)), None]
    xs = [_to_device(x_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    dys = [_to_device(dy_np[r * n_local:(r + 1) * n_local], dtype) for r in range(ranks)]
    gathered = torch.stack([bns.sync_local_moments(xs[r], sps[r], eps) for r in range(ranks)])
    mean, invstd, count = bns.sync_merge_moments(gathered, eps)
    ys = [bns.sync_normalize(xs[r], gamma, beta, mean, invstd) for r in range(ranks)]
    bns.sync_normalize(xv, gamma, beta, mean, invstd, y=sps[0].yv)
    partial = [bns.sync_backward_sums(xs[r], dys[r], gamma, mean, invstd, virtual_rows=sps[r]) for r in range(ranks)]
    sums = torch.stack([p[1] for p in partial]).sum(dim=0)
    dxs = [bns.sync_backward_apply(xs[r], dys[r], gamma, mean, invstd, sps[r], sums, count, partial[r][0])
           for r in range(ranks)]
    torch.cuda.synchronize()
    osp = O.Sampling.virtual(2)
    f = O.forward(x_np, gamma_np, beta_np, eps, osp, xv=xv_np)
    b = O.backward(x_np, dy_np, gamma_np, f.mean, f.var, eps, osp, xv=xv_np, dyv=dyv_np)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    tensor_close(np.concatenate([_to_host(t) for t in ys]), f.y, "y")
    close_f32(sps[0].yv.cpu().numpy(), f.yv, "yv")
    tensor_close(np.concatenate([_to_host(t) for t in dxs]), b.dx, "dx")
    close_f32(sps[0].dxv.cpu().numpy(), b.dxv, "dxv")
    close_f32(sums[0].cpu().numpy(), b.dbeta, "dbeta")
    close_f32(sums[1].cpu().numpy(), b.dgamma, "dgamma")


@pytest.mark.parametrize("rule,kw", [("batch", dict(k=5, contiguous=False)), ("batch", dict(k=4)),
                                     ("feature", dict(ph=3, pw=4, offset_mode=0)),
                                     ("feature", dict(ph=2, pw=2, offset_mode=2)), ("full", dict())])
@pytest.mark.parametrize("dtype,dims", [("f32", (24, 20, 14, 14)), ("bf16", (16, 24, 7, 7))])
@pytest.mark.parametrize("with_residual", [True, False])
def test_fused_residual_relu(rule, kw, dtype, dims, with_residual):
    """BN + residual + ReLU against the oracle's composition.  The rectifier's mask is a floating-point
    decision, so the case is drawn (deterministically) with every pre-activation away from zero by more
    than the two sides' rounding; then the masks agree and everything is compared element by element."""
    import torch
    from paper_1810_10962_b200 import bns
    from helpers import quantise
    for seed in range(96, 196):
        case = make_case(*dims, rule, seed=seed, dtype=dtype, **kw)
        res_np = quantise(I.upstream_gradient(case.x.shape, seed, I.TAG_XV), dtype) if with_residual else None
        osp = case.oracle_sampling()
        f = O.forward_relu(case.x, res_np, case.gamma, case.beta, case.eps, osp)
        if np.abs(f.z).min() > 2e-5:
            break
    else:
        pytest.fail("no seed keeps the pre-activations away from zero")
    b, dres_want = O.backward_relu(case.x, case.dy, case.gamma, f, case.eps, osp)
    x, dy = _to_device(case.x, dtype), _to_device(case.dy, dtype)
    res = _to_device(res_np, dtype) if with_residual else None
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    sp = gpu_sampling(case)
    y, mean, invstd = bns.forward_relu(x, res, gamma, beta, case.eps, sp)
    dx, dres, dgamma, dbeta = bns.backward_relu(x, res, dy, gamma, beta, mean, invstd, sp)
    torch.cuda.synchronize()
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    tensor_close(_to_host(y), f.y, "y")
    tensor_close(_to_host(dx), b.dx, "dx")
    close_f32(dgamma.cpu().numpy(), b.dgamma, "dgamma")
    close_f32(dbeta.cpu().numpy(), b.dbeta, "dbeta")
    if with_residual:
        assert np.array_equal(_to_host(dres), dres_want.astype(np.float32))     # dy or 0: bit-exact
    else:
        assert dres is None


def test_fused_residual_relu_at_benchmark_size():
    """The shape and rule that bench.py times as `fs_relu`: 256x64x56x56 fp32, 8x8 patch, with a residual.  At
    51 million elements some pre-activation always lands within rounding of zero, where the rectifier's mask
    is either side's to decide; so the residual is nudged, using the oracle's own pre-activations only, until
    every one of them is well away from zero.  Then the masks agree and every element is compared."""
    import torch
    from paper_1810_10962_b200 import bns
    case = make_case(256, 64, 56, 56, "feature", seed=98, ph=8, pw=8, offset_mode=0)
    osp = case.oracle_sampling()
    res_np = I.upstream_gradient(case.x.shape, 98, I.TAG_XV)
    f = O.forward_relu(case.x, res_np, case.gamma, case.beta, case.eps, osp)
    near = np.abs(f.z) < 1e-3
    res_np = np.where(near, res_np + np.float32(0.0625), res_np).astype(np.float32)
    f = O.forward_relu(case.x, res_np, case.gamma, case.beta, case.eps, osp)
    assert np.abs(f.z).min() > 5e-4
    b, dres_want = O.backward_relu(case.x, case.dy, case.gamma, f, case.eps, osp)
    x, dy, res = _to_device(case.x, "f32"), _to_device(case.dy, "f32"), _to_device(res_np, "f32")
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    sp = gpu_sampling(case)
    y, mean, invstd = bns.forward_relu(x, res, gamma, beta, case.eps, sp)
    dx, dres, dgamma, dbeta = bns.backward_relu(x, res, dy, gamma, beta, mean, invstd, sp)
    torch.cuda.synchronize()
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    close_f32(_to_host(y), f.y, "y")
    close_f32(_to_host(dx), b.dx, "dx")
    close_f32(dgamma.cpu().numpy(), b.dgamma, "dgamma")
    close_f32(dbeta.cpu().numpy(), b.dbeta, "dbeta")
    assert np.array_equal(_to_host(dres), dres_want.astype(np.float32))


def _nhwc(a):
    return np.ascontiguousarray(np.transpose(a, (0, 2, 3, 1)))


def _nchw(a):
    return np.ascontiguousarray(np.transpose(a, (0, 3, 1, 2)))


NHWC_CASES = [
    ("batch", dict(k=5, contiguous=False)), ("batch", dict(k=3)), ("feature", dict(ph=3, pw=4, offset_mode=0)),
    ("feature", dict(ph=2, pw=2, offset_mode=1)), ("feature", dict(ph=1, pw=1, offset_mode=0)),
    ("virtual", dict(nv=2)), ("virtual", dict(nv=1, with_dyv=False)), ("full", dict()),
]


@pytest.mark.parametrize("rule,kw", NHWC_CASES)
@pytest.mark.parametrize("dtype,dims", [("f32", (12, 64, 9, 11)), ("bf16", (10, 40, 7, 7)), ("f32", (6, 7, 5, 3)),
                                        ("bf16", (3, 2080, 2, 2)), ("f32", (40, 16, 16, 16))])
@pytest.mark.parametrize("direct_max", [0, 8192])
def test_channels_last_layout(rule, kw, dtype, dims, direct_max):
    """The NHWC entry points against the (NCHW) oracle on the transposed tensors; once with small sampled sets
    going through the one-block-per-strip kernels (the default) and once with every set going through partial
    sums and the finalize launches."""
    from paper_1810_10962_b200 import bns
    try:
        bns.set_tuning("direct_max", direct_max)
        _check_channels_last(rule, kw, dtype, dims)
    finally:
        bns.set_tuning("direct_max", 8192)


@pytest.mark.parametrize("rule,kw,dtype,dims", [
    ("batch", dict(k=32), "f32", (256, 64, 56, 56)),                            # bench.py --layout nhwc, first layer
    ("feature", dict(ph=8, pw=8, offset_mode=0), "f32", (256, 64, 56, 56)),     # ... and second: 802 816 rows
    ("feature", dict(ph=1, pw=1, offset_mode=0), "bf16", (256, 256, 14, 14)),   # a ResNet-50 layer
])
def test_channels_last_layout_at_benchmark_size(rule, kw, dtype, dims):
    _check_channels_last(rule, kw, dtype, dims)


def _check_channels_last(rule, kw, dtype, dims):
    import torch
    from paper_1810_10962_b200 import bns
    kw = dict(kw)
    N, C, H, W = dims
    if rule == "batch":
        kw["k"] = min(kw["k"], N)
    if rule == "feature":
        kw["ph"], kw["pw"] = min(kw["ph"], H), min(kw["pw"], W)
    if rule == "virtual":
        kw["xv_dtype"] = dtype
    case = make_case(N, C, H, W, rule, seed=97, dtype=dtype, **kw)
    dev = lambda a, d=dtype: _to_device(_nhwc(a), d)
    x, dy = dev(case.x), dev(case.dy)
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    if rule == "full":
        sp = bns.Sampling.full()
    elif rule == "batch":
        sp = bns.Sampling.batch(case.sample_idx)
    elif rule == "feature":
        off = case.offsets if case.offset_mode == 0 else torch.from_numpy(case.offsets).cuda()
        sp = bns.Sampling.feature(case.ph, case.pw, off, case.offset_mode)
    else:
        xv = dev(case.xv, case.xv_dtype)
        dyv = None if case.dyv is None else dev(case.dyv, case.xv_dtype)
        sp = bns.Sampling.virtual(xv, yv=torch.empty_like(xv), dyv=dyv, dxv=torch.empty_like(xv))
    y, mean, invstd, ws = bns.forward_nhwc(x, gamma, beta, case.eps, sp)
    dx, dgamma, dbeta = bns.backward_nhwc(x, dy, gamma, mean, invstd, sp, ws)
    torch.cuda.synchronize()
    from helpers import run_oracle
    f, b = run_oracle(case)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.cpu().numpy(), f.mean, "mean")
    close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
    tensor_close(_nchw(_to_host(y)), f.y, "y")
    tensor_close(_nchw(_to_host(dx)), b.dx, "dx")
    close_f32(dgamma.cpu().numpy(), b.dgamma, "dgamma")
    close_f32(dbeta.cpu().numpy(), b.dbeta, "dbeta")
    if rule == "virtual":
        tensor_close(_nchw(_to_host(sp.yv)), f.yv, "yv")
        tensor_close(_nchw(_to_host(sp.dxv)), b.dxv, "dxv")


def test_channels_last_rejects_per_map_offsets():
    import torch
    from paper_1810_10962_b200 import bns
    x = torch.zeros(2, 4, 4, 8, device="cuda")
    off = torch.zeros(2 * 8, 2, dtype=torch.int32, device="cuda")
    g = torch.ones(8, device="cuda")
    with pytest.raises(bns.BnsError):
        bns.forward_nhwc(x, g, g, 1e-5, bns.Sampling.feature(2, 2, off, bns.OFF_PER_MAP))
