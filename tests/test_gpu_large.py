"""GPU parity at the upper end of the supported sizes: a tensor of more than 2^32 elements, so that element
offsets of the last rows need 64 bits.  The tensors are drawn on the device (seeded); the oracle checks a few
whole channels, which it can do one by one because channels are independent."""
import numpy as np
import pytest

import oracle as O
from helpers import Case, GpuResult, _to_host, compare

pytestmark = pytest.mark.gpu

N, C, H, W = 300, 256, 250, 250          # 4.8e9 elements: the offsets of rows 269..299 do not fit 32 bits
CHECKED = [0, 101, 255]
NEED_BYTES = 56e9                        # four bf16 tensors of 9.6 GB and the transposes of the channels-last case


def _draw(shape, seed, channel_axis, channel_offsets):
    """Seeded N(0,1) values, bf16, filled in slices of the first axis; with `channel_offsets` plus a per-channel
    offset in [-1, 1] (activations).  The upstream gradient stays zero-mean: with 1.9e7 elements per channel a
    gradient of mean 1 would make sum dy (x - mean) move by 0.8 for the last bit of an fp32 mean, which says
    nothing about the kernels."""
    import torch
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    view = [1, 1, 1, 1]
    view[channel_axis] = shape[channel_axis]
    offset = torch.linspace(-1.0, 1.0, shape[channel_axis], device="cuda").view(view).to(torch.bfloat16)
    for n0 in range(0, shape[0], 25):
        t[n0:n0 + 25].normal_(generator=g)
        if channel_offsets:
            t[n0:n0 + 25].add_(offset)
    return t


def _channel_case(rule, x, dy, gamma, beta, c, nhwc, **kw):
    """The layer restricted to channel c, as host arrays for the oracle."""
    pick = (lambda t: t[..., c]) if nhwc else (lambda t: t[:, c])
    xs = _to_host(pick(x).contiguous()).reshape(N, 1, H, W)
    dys = _to_host(pick(dy).contiguous()).reshape(N, 1, H, W)
    return Case(xs, dys, gamma[c:c + 1].cpu().numpy(), beta[c:c + 1].cpu().numpy(), "bf16", rule,
                name=f"large-{rule}-{'nhwc' if nhwc else 'nchw'}-c{c}", **kw)


def _channel_result(y, mean, invstd, dx, dgamma, dbeta, c, nhwc):
    pick = (lambda t: t[..., c]) if nhwc else (lambda t: t[:, c])
    one = lambda v: v[c:c + 1].cpu().numpy()
    return GpuResult(_to_host(pick(y).contiguous()).reshape(N, 1, H, W), one(mean), one(invstd),
                     _to_host(pick(dx).contiguous()).reshape(N, 1, H, W), one(dgamma), one(dbeta))


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("rule", ["batch", "feature"])
def test_tensor_of_more_than_2_to_32_elements(rule, layout):
    import torch
    from paper_1810_10962_b200 import bns
    free, _ = torch.cuda.mem_get_info()
    if free < NEED_BYTES:
        pytest.skip(f"needs {NEED_BYTES / 1e9:.0f} GB of free device memory")
    assert N * C * H * W > 2 ** 32
    nhwc = layout == "nhwc"
    shape = (N, H, W, C) if nhwc else (N, C, H, W)
    x = _draw(shape, 1816, 3 if nhwc else 1, channel_offsets=True)
    dy = _draw(shape, 1817, 3 if nhwc else 1, channel_offsets=False)
    gamma = torch.linspace(0.5, 1.5, C, device="cuda")
    beta = torch.linspace(-0.1, 0.1, C, device="cuda")
    if rule == "batch":
        idx = np.array([299, 5, 280, 150, 271], dtype=np.int32)      # scattered, three of them beyond 2^32 elements
        sp, kw = bns.Sampling.batch(idx), dict(sample_idx=idx)
    else:
        off = np.array([H - 31, W - 31], dtype=np.int32)             # the patch in the last rows and columns of each map
        sp, kw = bns.Sampling.feature(31, 31, off, bns.OFF_SHARED), dict(ph=31, pw=31, offset_mode=0, offsets=off)
    if nhwc:
        y, mean, invstd, ws = bns.forward_nhwc(x, gamma, beta, 1e-5, sp)
        dx, dgamma, dbeta = bns.backward_nhwc(x, dy, gamma, mean, invstd, sp, ws)
    else:
        ws = bns.new_workspace(x, sp)
        y, mean, invstd = bns.forward(x, gamma, beta, 1e-5, sp, workspace=ws)
        dx, dgamma, dbeta = bns.backward(x, dy, gamma, mean, invstd, sp, workspace=ws)
    torch.cuda.synchronize()
    assert bns.wait_timeouts() == 0
    for c in CHECKED:
        case = _channel_case(rule, x, dy, gamma, beta, c, nhwc, **kw)
        compare(case, _channel_result(y, mean, invstd, dx, dgamma, dbeta, c, nhwc))
    del x, dy, y, dx
    torch.cuda.empty_cache()
