"""Shared machinery of the GPU parity tests: build a seeded case, run it through the C ABI (via the
Python binding) and through the CPU oracle, and compare element by element."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

import bns_inputs as I
import oracle as O

EPS = 1e-5


@dataclass
class Case:
    """Inputs of one layer, as float32 numpy arrays whose values are exactly representable in
    `dtype` (so the oracle and the GPU start from identical numbers)."""
    x: np.ndarray
    dy: np.ndarray
    gamma: np.ndarray
    beta: np.ndarray
    dtype: str                      # "f32" | "bf16"
    rule: str                       # "full" | "batch" | "feature" | "virtual"
    sample_idx: Optional[np.ndarray] = None
    ph: int = 0
    pw: int = 0
    offset_mode: int = 0
    offsets: Optional[np.ndarray] = None
    xv: Optional[np.ndarray] = None
    dyv: Optional[np.ndarray] = None
    xv_dtype: str = "f32"
    eps: float = EPS
    name: str = ""

    def oracle_sampling(self) -> O.Sampling:
        if self.rule == "full":
            return O.Sampling.full()
        if self.rule == "batch":
            return O.Sampling.batch(self.sample_idx)
        if self.rule == "feature":
            return O.Sampling.feature(self.ph, self.pw, self.offsets, self.offset_mode)
        return O.Sampling.virtual(self.xv.shape[0])


def quantise(a: np.ndarray, dtype: str) -> np.ndarray:
    return I.round_to_bf16(a) if dtype == "bf16" else np.ascontiguousarray(a, dtype=np.float32)


def make_case(N, C, H, W, rule, seed, dtype="f32", generator="correlated", k=2, contiguous=True, ph=2, pw=2,
              offset_mode=0, nv=2, xv_dtype="f32", with_dyv=True, name="") -> Case:
    gen = I.correlated_activations if generator == "correlated" else I.tiny_activations
    x = quantise(gen(N, C, H, W, seed), dtype)
    dy = quantise(I.upstream_gradient(x.shape, seed), dtype)
    gamma, beta = I.affine_parameters(C, seed)
    case = Case(x, dy, gamma, beta, dtype, rule, name=name or f"{rule}-{dtype}-{N}x{C}x{H}x{W}")
    if rule == "batch":
        case.sample_idx = I.batch_sample_indices(N, k, seed, contiguous)
    elif rule == "feature":
        case.ph, case.pw, case.offset_mode = ph, pw, offset_mode
        case.offsets = I.patch_offsets(N, C, H, W, ph, pw, offset_mode, seed)
    elif rule == "virtual":
        case.xv_dtype = xv_dtype
        case.xv = quantise(I.virtual_samples(nv, C, H, W, seed), xv_dtype)
        case.dyv = quantise(I.upstream_gradient(case.xv.shape, seed, I.TAG_DYV), xv_dtype) if with_dyv else None
    return case


# ----------------------------------------------------------------------------- GPU side
def _to_device(a: np.ndarray, dtype: str):
    import torch
    if dtype == "bf16":
        bits = I.f32_to_bf16_bits(a)          # exact: the values are already bf16-representable
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _to_host(t) -> np.ndarray:
    import torch
    if t.dtype == torch.bfloat16:
        return I.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


@dataclass
class GpuResult:
    y: np.ndarray
    mean: np.ndarray
    invstd: np.ndarray
    dx: np.ndarray
    dgamma: np.ndarray
    dbeta: np.ndarray
    yv: Optional[np.ndarray] = None
    dxv: Optional[np.ndarray] = None
    raw: dict = field(default_factory=dict)   # device tensors, for bit-exact run-to-run comparison


def gpu_sampling(case: Case):
    import torch
    from paper_1810_10962_b200 import bns
    if case.rule == "full":
        return bns.Sampling.full()
    if case.rule == "batch":
        return bns.Sampling.batch(case.sample_idx)
    if case.rule == "feature":
        off = case.offsets
        if case.offset_mode != bns.OFF_SHARED:
            off = torch.from_numpy(np.ascontiguousarray(off, dtype=np.int32)).cuda()
        return bns.Sampling.feature(case.ph, case.pw, off, case.offset_mode)
    xv = _to_device(case.xv, case.xv_dtype)
    dyv = None if case.dyv is None else _to_device(case.dyv, case.xv_dtype)
    return bns.Sampling.virtual(xv, yv=torch.empty_like(xv), dyv=dyv, dxv=torch.empty_like(xv))


def run_gpu(case: Case, use_full_bn_entry=False) -> GpuResult:
    import torch
    from paper_1810_10962_b200 import bns
    x, dy = _to_device(case.x, case.dtype), _to_device(case.dy, case.dtype)
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    sp = gpu_sampling(case)
    ws = bns.new_workspace(x, sp)
    if use_full_bn_entry:
        assert case.rule == "full"
        y, mean, invstd = bns.full_bn(x, gamma, beta, case.eps, workspace=ws)
    else:
        y, mean, invstd = bns.forward(x, gamma, beta, case.eps, sp, workspace=ws)
    dx, dgamma, dbeta = bns.backward(x, dy, gamma, mean, invstd, sp, workspace=ws)
    torch.cuda.synchronize()
    assert bns.wait_timeouts() == 0, "a bounded wait of a kernel ran out"
    res = GpuResult(_to_host(y), mean.cpu().numpy(), invstd.cpu().numpy(), _to_host(dx), dgamma.cpu().numpy(),
                    dbeta.cpu().numpy(), raw=dict(y=y, mean=mean, invstd=invstd, dx=dx, dgamma=dgamma, dbeta=dbeta))
    if case.rule == "virtual":
        res.yv, res.dxv = _to_host(sp.yv), _to_host(sp.dxv)
        res.raw.update(yv=sp.yv, dxv=sp.dxv)
    return res


# ----------------------------------------------------------------------------- oracle side and comparison
def run_oracle(case: Case, channels=None):
    sp = case.oracle_sampling()
    f = O.forward(case.x, case.gamma, case.beta, case.eps, sp, xv=case.xv, channels=channels)
    b = O.backward(case.x, case.dy, case.gamma, f.mean, f.var, case.eps, sp, xv=case.xv, dyv=case.dyv,
                   channels=channels)
    return f, b


def close_f32(got, want, what, atol=1e-4, rtol=1e-4):
    """fp32 bar: |g - o| <= 1e-4 + 1e-4 |o| element-wise."""
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - want)
    bound = atol + rtol * np.abs(want)
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} outside 1e-4/1e-4; worst |err|="
                           f"{err.max():.3e} at {np.unravel_index(np.argmax(err - bound), err.shape)}")


def close_bf16(got, want, what, rel=2e-2):
    """bf16 bar: |g - o| <= 2e-2 max(|o|, 1) element-wise."""
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - want)
    bound = rel * np.maximum(np.abs(want), 1.0)
    bad = err > bound
    assert not bad.any(), f"{what}: {int(bad.sum())} of {bad.size} outside rel 2e-2; worst |err|={err.max():.3e}"


def compare(case: Case, g: GpuResult, channels=None):
    """Element-by-element comparison with the oracle (on `channels`, or on every channel)."""
    f, b = run_oracle(case, channels)
    sel = slice(None) if channels is None else np.asarray(channels)
    tensor_close = close_f32 if case.dtype == "f32" else close_bf16
    close_f32(g.mean[sel], f.mean, f"{case.name} mean")
    close_f32(g.invstd[sel], f.invstd, f"{case.name} invstd")
    tensor_close(g.y[:, sel], f.y, f"{case.name} y")
    tensor_close(g.dx[:, sel], b.dx, f"{case.name} dx")
    close_f32(g.dgamma[sel], b.dgamma, f"{case.name} dgamma")
    close_f32(g.dbeta[sel], b.dbeta, f"{case.name} dbeta")
    if case.rule == "virtual":
        v_close = close_f32 if case.xv_dtype == "f32" else close_bf16
        v_close(g.yv[:, sel], f.yv, f"{case.name} yv")
        v_close(g.dxv[:, sel], b.dxv, f"{case.name} dxv")
    return f, b
