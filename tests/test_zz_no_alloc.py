"""bns_forward_static: the forward for callers that are not allowed to allocate device memory
(plug-ins inside a server that owns the whole device pool, code paths where cudaMalloc would stall
other tenants' streams).  It must give what bns_forward gives, call after call, although all calls
share one built-in scratch array that still holds the previous call's partial sums."""
import numpy as np
import pytest

import oracle as O
from helpers import _to_device, _to_host, close_bf16, close_f32, gpu_sampling, make_case


@pytest.mark.gpu
def test_forward_static_matches_forward_on_two_calls_in_a_row():
    import torch
    from paper_1810_10962_b200 import bns

    # two different layers back to back: the second call finds the first one's leftovers in the scratch.
    # The first goes through partial sums kept in the scratch (a large sampled set on a tensor above the
    # size that runs on chip), the second clears and uses the status word at its start.
    cases = [make_case(64, 32, 28, 28, "batch", seed=91, k=16),
             make_case(48, 24, 14, 14, "feature", seed=92, dtype="bf16", ph=3, pw=3, offset_mode=2)]
    for number, case in enumerate(cases):
        x = _to_device(case.x, case.dtype)
        gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
        sp = gpu_sampling(case)
        assert bns.workspace_bytes(x, sp) <= bns.static_workspace_bytes()
        if number == 0:
            assert bns.slab_plan(x, sp) is None          # the streaming kernels: this call needs its scratch
        want_y, want_mean, want_invstd = bns.forward(x, gamma, beta, case.eps, sp)
        # the caller owns every tensor it passes in, outputs included
        y = torch.empty_like(x)
        mean = torch.empty(x.shape[1], dtype=torch.float32, device="cuda")
        invstd = torch.empty_like(mean)
        bns.forward_static(x, gamma, beta, case.eps, sp, y, mean, invstd)      # first call on the device: looks up the array
        torch.cuda.synchronize()
        # ... and the call itself takes no device memory: the driver's count of free bytes does not move
        free_before, _ = torch.cuda.mem_get_info()
        bns.forward_static(x, gamma, beta, case.eps, sp, y, mean, invstd)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        # same results as the entry point with a caller-provided workspace, within the tolerances of the parity tests
        np.testing.assert_allclose(mean.cpu().numpy(), want_mean.cpu().numpy(), rtol=1e-4, atol=1e-4)
        np.testing.assert_allclose(invstd.cpu().numpy(), want_invstd.cpu().numpy(), rtol=1e-4, atol=1e-4)
        tol = dict(rtol=1e-4, atol=1e-4) if case.dtype == "f32" else dict(rtol=2e-2, atol=2e-2)
        np.testing.assert_allclose(y.float().cpu().numpy(), want_y.float().cpu().numpy(), **tol)
        # and the same as the oracle
        f = O.forward(case.x, case.gamma, case.beta, case.eps, case.oracle_sampling())
        close_f32(mean.cpu().numpy(), f.mean, "mean")
        close_f32(invstd.cpu().numpy(), f.invstd, "invstd")
        (close_f32 if case.dtype == "f32" else close_bf16)(_to_host(y), f.y, "y")


@pytest.mark.gpu
def test_forward_static_rejects_what_does_not_fit():
    import torch
    from paper_1810_10962_b200 import bns
    # N=256, C=8192, 7x7 bf16 needs more scratch than is built in: refused on the host, nothing launched.
    # Real tensors all the same, so that a check that stopped working could not send a kernel to a wild address.
    x = torch.zeros(256, 8192, 7, 7, dtype=torch.bfloat16, device="cuda")
    y = torch.empty_like(x)
    vec = [torch.ones(8192, device="cuda") for _ in range(4)]
    sp = bns.Sampling.feature(1, 1, np.array([0, 0]))
    assert bns.workspace_bytes(x, sp) > bns.static_workspace_bytes()
    with pytest.raises(bns.BnsError) as err:
        bns.forward_static(x, vec[0], vec[1], 1e-5, sp, y, vec[2], vec[3])
    assert err.value.status == -7
