"""bns_forward_static: the forward for callers that are not allowed to allocate device memory
(plug-ins inside a server that owns the whole device pool, code paths where cudaMalloc would stall
other tenants' streams).  It must give what bns_forward gives, call after call, although all calls
share one built-in scratch array that still holds the previous call's partial sums."""
import numpy as np
import pytest

from helpers import _to_device, gpu_sampling, make_case


@pytest.mark.gpu
def test_forward_static_matches_forward_on_two_calls_in_a_row():
    import torch
    from paper_1810_10962_b200 import bns

    # two different layers back to back: the second call finds the first one's leftovers in the scratch
    cases = [make_case(64, 32, 28, 28, "batch", seed=91, k=8),
             make_case(48, 24, 14, 14, "feature", seed=92, dtype="bf16", ph=3, pw=3, offset_mode=2)]
    for case in cases:
        x = _to_device(case.x, case.dtype)
        gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
        sp = gpu_sampling(case)
        assert bns.workspace_bytes(x, sp) <= bns.static_workspace_bytes()
        want_y, want_mean, want_invstd = bns.forward(x, gamma, beta, case.eps, sp)
        # the caller owns every tensor it passes in, outputs included; the call itself allocates nothing
        y = torch.empty_like(x)
        mean = torch.empty(x.shape[1], dtype=torch.float32, device="cuda")
        invstd = torch.empty_like(mean)
        bns.forward_static(x, gamma, beta, case.eps, sp, y, mean, invstd)
        torch.cuda.synchronize()
        np.testing.assert_allclose(mean.cpu().numpy(), want_mean.cpu().numpy(), rtol=1e-4, atol=1e-4)
        np.testing.assert_allclose(invstd.cpu().numpy(), want_invstd.cpu().numpy(), rtol=1e-4, atol=1e-4)
        tol = dict(rtol=1e-4, atol=1e-4) if case.dtype == "f32" else dict(rtol=2e-2, atol=2e-2)
        np.testing.assert_allclose(y.float().cpu().numpy(), want_y.float().cpu().numpy(), **tol)


@pytest.mark.gpu
def test_forward_static_rejects_what_does_not_fit():
    import ctypes
    from paper_1810_10962_b200 import bns
    lib = bns.load()
    # N=256, C=8192, 7x7 bf16 needs more scratch than is built in: refused on the host, nothing launched
    sh = bns._Shape(256, 8192, 7, 7, bns.BF16)
    sp = bns.Sampling.feature(1, 1, np.array([0, 0]))._c()
    assert lib.bns_workspace_bytes(ctypes.byref(sh), ctypes.byref(sp)) > bns.static_workspace_bytes()
    st = lib.bns_forward_static(ctypes.byref(sh), 0x1000, 0x2000, 0x3000, 1e-5, ctypes.byref(sp), 0x4000, 0x5000,
                                0x6000, None)
    assert st == -7
