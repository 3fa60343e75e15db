"""Python binding of the C ABI in ``include/bns.h``.

Argument marshalling only: every function hands raw device pointers, sizes and the current CUDA
stream to ``libbns.so``; all arithmetic runs in that library's kernels.  PyTorch provides device
memory and streams.  There is no fallback: if the library cannot be loaded, or a tensor is not a
CUDA tensor, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import build as _build

OK = 0
F32, BF16 = 0, 1
RULE_FULL, RULE_BATCH, RULE_FEATURE, RULE_VIRTUAL = 0, 1, 2, 3
OFF_SHARED, OFF_PER_SAMPLE, OFF_PER_MAP = 0, 1, 2
FLAG_BAD_OFFSET = 1

KERNEL_KINDS = 14
(KERNEL_COL_MOMENTS, KERNEL_PATCH_MOMENTS, KERNEL_FINALIZE_STATS, KERNEL_NORMALIZE, KERNEL_BWD_REDUCE,
 KERNEL_FINALIZE_BWD, KERNEL_COL_FIXUP, KERNEL_PATCH_FIXUP, KERNEL_MASK, KERNEL_DIRECT_MOMENTS,
 KERNEL_DIRECT_FIXUP, KERNEL_VECTOR, KERNEL_SLAB_FORWARD, KERNEL_SLAB_BACKWARD) = range(KERNEL_KINDS)

EXPORTS = [
    "bns_workspace_bytes", "bns_forward", "bns_forward_static", "bns_static_workspace_bytes", "bns_backward", "bns_full_bn", "bns_host_arena_bytes",
    "bns_forward_backward_host", "bns_debug_selection_mask", "bns_workspace_status", "bns_status_string",
    "bns_launch_count", "bns_launch_count_reset", "bns_profile_enable", "bns_profile_read", "bns_kernel_name",
    "bns_set_tuning", "bns_slab_plan", "bns_wait_timeouts",
    "bns_workspace_bytes_mixed", "bns_forward_mixed", "bns_backward_mixed", "bns_update_moving_average",
    "bns_inference_forward", "bns_forward_training",
    "bns_sync_local_moments", "bns_sync_merge_moments", "bns_sync_normalize", "bns_sync_backward_sums",
    "bns_sync_backward_apply",
    "bns_forward_relu", "bns_backward_relu",
    "bns_workspace_bytes_nhwc", "bns_forward_nhwc", "bns_backward_nhwc",
]


class BnsError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


class _Shape(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int), ("C", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int),
                ("dtype", ctypes.c_int)]


class _Sampling(ctypes.Structure):
    _fields_ = [
        ("rule", ctypes.c_int), ("k", ctypes.c_int), ("sample_idx", ctypes.c_void_p),
        ("ph", ctypes.c_int), ("pw", ctypes.c_int), ("offset_mode", ctypes.c_int), ("offsets", ctypes.c_void_p),
        ("nv", ctypes.c_int), ("xv_dtype", ctypes.c_int), ("xv", ctypes.c_void_p), ("yv", ctypes.c_void_p),
        ("dyv", ctypes.c_void_p), ("dxv", ctypes.c_void_p),
    ]


_lib = None


def library_path() -> str:
    return _build.LIBRARY


def load():
    """Load ``libbns.so`` (building it first if its sources are newer and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    if _build.is_stale():
        try:
            _build.build()
        except Exception as exc:  # no compiler: only acceptable if a built library is already there
            if not os.path.exists(_build.LIBRARY):
                raise RuntimeError(f"libbns.so is missing and could not be built: {exc}") from exc
    lib = ctypes.CDLL(_build.LIBRARY)
    vp, sz, fl = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float
    shp, smp = ctypes.POINTER(_Shape), ctypes.POINTER(_Sampling)
    lib.bns_workspace_bytes.restype = sz
    lib.bns_workspace_bytes.argtypes = [shp, smp]
    lib.bns_forward.restype = ctypes.c_int
    lib.bns_forward.argtypes = [shp, vp, vp, vp, fl, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_forward_static.restype = ctypes.c_int
    lib.bns_forward_static.argtypes = [shp, vp, vp, vp, fl, smp, vp, vp, vp, vp]
    lib.bns_static_workspace_bytes.restype = sz
    lib.bns_static_workspace_bytes.argtypes = []
    lib.bns_backward.restype = ctypes.c_int
    lib.bns_backward.argtypes = [shp, vp, vp, vp, vp, vp, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_full_bn.restype = ctypes.c_int
    lib.bns_full_bn.argtypes = [shp, vp, vp, vp, fl, vp, vp, vp, vp, sz, vp]
    lib.bns_host_arena_bytes.restype = sz
    lib.bns_host_arena_bytes.argtypes = [shp, smp]
    lib.bns_forward_backward_host.restype = ctypes.c_int
    lib.bns_forward_backward_host.argtypes = [shp, vp, vp, vp, vp, fl, smp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.bns_debug_selection_mask.restype = ctypes.c_int
    lib.bns_debug_selection_mask.argtypes = [shp, smp, vp, vp, sz, vp]
    lib.bns_workspace_status.restype = ctypes.c_int
    lib.bns_workspace_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    lib.bns_status_string.restype = ctypes.c_char_p
    lib.bns_status_string.argtypes = [ctypes.c_int]
    lib.bns_launch_count.restype = ctypes.c_uint64
    lib.bns_launch_count_reset.restype = None
    lib.bns_profile_enable.restype = None
    lib.bns_profile_enable.argtypes = [ctypes.c_int]
    lib.bns_profile_read.restype = ctypes.c_int
    lib.bns_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)]
    lib.bns_kernel_name.restype = ctypes.c_char_p
    lib.bns_kernel_name.argtypes = [ctypes.c_int]
    lib.bns_workspace_bytes_mixed.restype = sz
    lib.bns_workspace_bytes_mixed.argtypes = [shp, smp]
    lib.bns_forward_mixed.restype = ctypes.c_int
    lib.bns_forward_mixed.argtypes = [shp, vp, vp, vp, fl, fl, smp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.bns_backward_mixed.restype = ctypes.c_int
    lib.bns_backward_mixed.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, fl, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_update_moving_average.restype = ctypes.c_int
    lib.bns_update_moving_average.argtypes = [ctypes.c_int, vp, vp, fl, fl, ctypes.c_int, vp, vp, vp]
    lib.bns_forward_training.restype = ctypes.c_int
    lib.bns_forward_training.argtypes = [shp, vp, vp, vp, fl, smp, fl, ctypes.c_int, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.bns_inference_forward.restype = ctypes.c_int
    lib.bns_inference_forward.argtypes = [shp, vp, vp, vp, fl, vp, vp, vp, vp, sz, vp]
    lib.bns_sync_local_moments.restype = ctypes.c_int
    lib.bns_sync_local_moments.argtypes = [shp, vp, smp, fl, vp, vp, sz, vp]
    lib.bns_sync_merge_moments.restype = ctypes.c_int
    lib.bns_sync_merge_moments.argtypes = [ctypes.c_int, ctypes.c_int, vp, fl, vp, vp, vp, vp]
    lib.bns_sync_normalize.restype = ctypes.c_int
    lib.bns_sync_normalize.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp]
    lib.bns_sync_backward_sums.restype = ctypes.c_int
    lib.bns_sync_backward_sums.argtypes = [shp, vp, vp, vp, vp, vp, smp, vp, vp, vp, sz, vp]
    lib.bns_sync_backward_apply.restype = ctypes.c_int
    lib.bns_sync_backward_apply.argtypes = [shp, vp, vp, vp, vp, vp, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_forward_relu.restype = ctypes.c_int
    lib.bns_forward_relu.argtypes = [shp, vp, vp, vp, vp, fl, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_backward_relu.restype = ctypes.c_int
    lib.bns_backward_relu.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, smp, vp, vp, vp, vp, vp, sz, vp]
    lib.bns_workspace_bytes_nhwc.restype = sz
    lib.bns_workspace_bytes_nhwc.argtypes = [shp, smp]
    lib.bns_forward_nhwc.restype = ctypes.c_int
    lib.bns_forward_nhwc.argtypes = [shp, vp, vp, vp, fl, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_backward_nhwc.restype = ctypes.c_int
    lib.bns_backward_nhwc.argtypes = [shp, vp, vp, vp, vp, vp, smp, vp, vp, vp, vp, sz, vp]
    lib.bns_set_tuning.restype = ctypes.c_int
    lib.bns_set_tuning.argtypes = [ctypes.c_char_p, ctypes.c_int]
    lib.bns_slab_plan.restype = ctypes.c_int
    lib.bns_slab_plan.argtypes = [shp, smp, ctypes.c_int, ctypes.POINTER(ctypes.c_int32)]
    lib.bns_wait_timeouts.restype = ctypes.c_int
    lib.bns_wait_timeouts.argtypes = [ctypes.POINTER(ctypes.c_uint32), vp]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().bns_status_string(int(status)).decode()


# ----------------------------------------------------------------------------- sampling rule
@dataclass
class Sampling:
    """The sampled set S.  ``sample_idx`` is a host int32 array; ``offsets`` is a host array for the
    shared location and a CUDA int32 tensor [N,2] / [N*C,2] otherwise; xv, yv, dyv, dxv are CUDA
    tensors [nv,C,H,W]."""
    rule: int = RULE_FULL
    sample_idx: Optional[np.ndarray] = None
    ph: int = 0
    pw: int = 0
    offset_mode: int = OFF_SHARED
    offsets: object = None
    nv: int = 0
    xv: Optional[torch.Tensor] = None
    yv: Optional[torch.Tensor] = None
    dyv: Optional[torch.Tensor] = None
    dxv: Optional[torch.Tensor] = None

    @staticmethod
    def full():
        return Sampling(RULE_FULL)

    @staticmethod
    def batch(sample_idx):
        return Sampling(RULE_BATCH, sample_idx=np.ascontiguousarray(sample_idx, dtype=np.int32))

    @staticmethod
    def feature(ph, pw, offsets, offset_mode=OFF_SHARED):
        if offset_mode == OFF_SHARED:
            offsets = np.ascontiguousarray(np.asarray(offsets).reshape(-1), dtype=np.int32)
        return Sampling(RULE_FEATURE, ph=int(ph), pw=int(pw), offset_mode=int(offset_mode), offsets=offsets)

    @staticmethod
    def virtual(xv, yv=None, dyv=None, dxv=None):
        return Sampling(RULE_VIRTUAL, nv=int(xv.shape[0]), xv=xv, yv=yv, dyv=dyv, dxv=dxv)

    def with_virtual(self, xv, yv=None, dyv=None, dxv=None):
        """This BATCH / FEATURE rule combined with virtual samples (for forward_mixed / backward_mixed)."""
        return Sampling(self.rule, sample_idx=self.sample_idx, ph=self.ph, pw=self.pw, offset_mode=self.offset_mode,
                        offsets=self.offsets, nv=int(xv.shape[0]), xv=xv, yv=yv, dyv=dyv, dxv=dxv)

    def _c(self, shape=None) -> _Sampling:
        """The C struct.  With `shape` (the _Shape of x) the length of device-resident patch offsets is
        checked against it: the kernels index them by sample (and channel), so a shorter tensor would be
        read out of bounds."""
        c = _Sampling()
        c.rule = self.rule
        if self.rule == RULE_BATCH:
            c.k = int(self.sample_idx.size)
            c.sample_idx = self.sample_idx.ctypes.data
        elif self.rule == RULE_FEATURE:
            c.ph, c.pw, c.offset_mode = self.ph, self.pw, self.offset_mode
            if self.offset_mode == OFF_SHARED:
                c.offsets = self.offsets.ctypes.data
            else:
                off = self.offsets
                if not (isinstance(off, torch.Tensor) and off.is_cuda and off.dtype == torch.int32 and off.is_contiguous()):
                    raise TypeError("per-sample / per-map offsets must be a contiguous CUDA int32 tensor")
                if shape is not None:
                    pairs = shape.N if self.offset_mode == OFF_PER_SAMPLE else shape.N * shape.C
                    if off.numel() != 2 * pairs:
                        raise TypeError(f"offsets must hold {pairs} (oh, ow) pairs for this shape and offset mode, "
                                        f"got {off.numel()} int32 values")
                c.offsets = off.data_ptr()
        if self.xv is not None:      # the VIRTUAL rule, or a sampling rule combined with virtual samples (Eq. 4)
            c.nv = int(self.xv.shape[0])
            c.xv_dtype = _dtype_code(self.xv)
            c.xv = _dev(self.xv)
            for name in ("yv", "dyv", "dxv"):
                t = getattr(self, name)
                if t is not None:
                    if t.dtype != self.xv.dtype or t.shape != self.xv.shape:
                        raise TypeError(f"{name} must match xv in dtype and shape")
                    setattr(c, name, _dev(t))
        return c


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported element type {t.dtype}")


def _dev(t: torch.Tensor) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("expected a CUDA tensor (this library has no CPU path)")
    if not t.is_contiguous():
        raise TypeError("expected a contiguous tensor")
    return t.data_ptr()


def _like(t: torch.Tensor, x: torch.Tensor, name: str) -> int:
    """Device pointer of a tensor that must match x in shape and element type (outputs are written in full)."""
    if t.shape != x.shape or t.dtype != x.dtype:
        raise TypeError(f"{name} must have the shape and dtype of x")
    return _dev(t)


def _check_virtual(x: torch.Tensor, sampling) -> None:
    """Virtual samples are [nv, ...] with the per-sample shape of x (same layout)."""
    if sampling.xv is not None and tuple(sampling.xv.shape[1:]) != tuple(x.shape[1:]):
        raise TypeError("xv must have the per-sample shape of x")


def _vec(t: torch.Tensor, C: int) -> int:
    if t.dtype != torch.float32 or t.numel() != C:
        raise TypeError("per-channel vectors must be float32 of length C")
    return _dev(t)


def _shape(x: torch.Tensor) -> _Shape:
    if x.dim() != 4:
        raise TypeError("expected an NCHW tensor")
    N, C, H, W = x.shape
    return _Shape(N, C, H, W, _dtype_code(x))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, what: str):
    if status != OK:
        raise BnsError(status, what)


def workspace_bytes(x: torch.Tensor, sampling: Sampling) -> int:
    sh = _shape(x)
    sp = sampling._c(sh)
    n = load().bns_workspace_bytes(ctypes.byref(sh), ctypes.byref(sp))
    if n == 0:
        raise BnsError(-3, "bns_workspace_bytes (invalid shape or sampling rule)")
    return int(n)


def new_workspace(x: torch.Tensor, sampling: Sampling) -> torch.Tensor:
    """Allocate a workspace for this shape and rule."""
    return torch.empty(workspace_bytes(x, sampling), dtype=torch.uint8, device=x.device)


def _workspace(x, sampling, workspace):
    if workspace is None:
        workspace = new_workspace(x, sampling)
    return workspace, workspace.data_ptr(), workspace.numel()


# ----------------------------------------------------------------------------- the three calls
def forward(x, gamma, beta, eps, sampling: Sampling, y=None, mean=None, invstd=None, workspace=None):
    """bns_forward: returns (y, mean, invstd)."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    mean = torch.empty(C, dtype=torch.float32, device=x.device) if mean is None else mean
    invstd = torch.empty(C, dtype=torch.float32, device=x.device) if invstd is None else invstd
    ws, wp, wn = _workspace(x, sampling, workspace)
    st = load().bns_forward(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps), ctypes.byref(sp),
                            _like(y, x, "y"), _vec(mean, C), _vec(invstd, C), wp, wn, _stream())
    _check(st, "bns_forward")
    return y, mean, invstd


def forward_training(x, gamma, beta, eps, sampling: Sampling, alpha, first_iteration, mean_ma, var_ma, y=None,
                     workspace=None):
    """bns_forward_training: bns_forward that also updates the moving averages of Eq. 8 in place.
    Returns (y, mean, invstd)."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    mean, invstd = (torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    ws, wp, wn = _workspace(x, sampling, workspace)
    st = load().bns_forward_training(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps), ctypes.byref(sp),
                                     float(alpha), 1 if first_iteration else 0, _vec(mean_ma, C), _vec(var_ma, C),
                                     _like(y, x, "y"), _vec(mean, C), _vec(invstd, C), wp, wn, _stream())
    _check(st, "bns_forward_training")
    return y, mean, invstd


def static_workspace_bytes() -> int:
    return int(load().bns_static_workspace_bytes())


def forward_static(x, gamma, beta, eps, sampling: Sampling, y, mean, invstd):
    """bns_forward_static: the forward for callers that may not allocate device memory.  The caller
    passes every tensor, outputs included; the scratch is the array built into the library, shared by
    all calls on the device (so do not overlap two of them).  Returns (y, mean, invstd)."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    st = load().bns_forward_static(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps),
                                   ctypes.byref(sp), _like(y, x, "y"), _vec(mean, C), _vec(invstd, C), _stream())
    _check(st, "bns_forward_static")
    return y, mean, invstd


def backward(x, dy, gamma, mean, invstd, sampling: Sampling, dx=None, dgamma=None, dbeta=None, workspace=None):
    """bns_backward: returns (dx, dgamma, dbeta)."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    if dy.shape != x.shape or dy.dtype != x.dtype:
        raise TypeError("dy must match x")
    dx = torch.empty_like(x) if dx is None else dx
    dgamma = torch.empty(C, dtype=torch.float32, device=x.device) if dgamma is None else dgamma
    dbeta = torch.empty(C, dtype=torch.float32, device=x.device) if dbeta is None else dbeta
    ws, wp, wn = _workspace(x, sampling, workspace)
    st = load().bns_backward(ctypes.byref(sh), _dev(x), _dev(dy), _vec(gamma, C), _vec(mean, C), _vec(invstd, C),
                             ctypes.byref(sp), _like(dx, x, "dx"), _vec(dgamma, C), _vec(dbeta, C), wp, wn, _stream())
    _check(st, "bns_backward")
    return dx, dgamma, dbeta


def full_bn(x, gamma, beta, eps, y=None, mean=None, invstd=None, workspace=None):
    """bns_full_bn: ordinary BN forward; returns (y, mean, invstd)."""
    sh = _shape(x)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    mean = torch.empty(C, dtype=torch.float32, device=x.device) if mean is None else mean
    invstd = torch.empty(C, dtype=torch.float32, device=x.device) if invstd is None else invstd
    ws, wp, wn = _workspace(x, Sampling.full(), workspace)
    st = load().bns_full_bn(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps), _like(y, x, "y"),
                            _vec(mean, C), _vec(invstd, C), wp, wn, _stream())
    _check(st, "bns_full_bn")
    return y, mean, invstd


def selection_mask(x, sampling: Sampling, workspace=None):
    """bns_debug_selection_mask: uint8 [N,C,H,W]."""
    sh = _shape(x)
    sp = sampling._c(sh)
    mask = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    ws, wp, wn = _workspace(x, sampling, workspace)
    _check(load().bns_debug_selection_mask(ctypes.byref(sh), ctypes.byref(sp), mask.data_ptr(), wp, wn, _stream()),
           "bns_debug_selection_mask")
    return mask


def workspace_status(workspace: torch.Tensor) -> int:
    flags = ctypes.c_uint32(0)
    _check(load().bns_workspace_status(workspace.data_ptr(), ctypes.byref(flags), _stream()), "bns_workspace_status")
    return int(flags.value)


class Prepared:
    """One layer's forward/backward with the argument marshalling done once.

    For a training loop that calls the same layer on the same buffers every step: the ctypes structures
    and raw pointers are built here, and forward() / backward() only make the C call (on the CUDA stream
    that is current at call time).  The tensors are kept alive by this object."""

    def __init__(self, x, dy, gamma, beta, eps, sampling: Sampling, y, dx, mean, invstd, dgamma, dbeta, workspace,
                 full_bn_entry=False):
        C = x.shape[1]
        if dy.shape != x.shape or dy.dtype != x.dtype:
            raise TypeError("dy must match x")
        self._keep = (x, dy, gamma, beta, sampling, y, dx, mean, invstd, dgamma, dbeta, workspace)
        self._lib = load()
        self._sh = _shape(x)
        self._sp = sampling._c(self._sh)
        self._eps = float(eps)
        self._full = bool(full_bn_entry)
        self._x, self._dy, self._y, self._dx = _dev(x), _dev(dy), _like(y, x, "y"), _like(dx, x, "dx")
        self._gamma, self._beta = _vec(gamma, C), _vec(beta, C)
        self._mean, self._invstd = _vec(mean, C), _vec(invstd, C)
        self._dgamma, self._dbeta = _vec(dgamma, C), _vec(dbeta, C)
        self._ws, self._wn = workspace.data_ptr(), workspace.numel()
        if self._wn < workspace_bytes(x, sampling):
            raise BnsError(-7, "workspace too small")

    def forward(self):
        stream = torch.cuda.current_stream().cuda_stream
        if self._full:
            st = self._lib.bns_full_bn(ctypes.byref(self._sh), self._x, self._gamma, self._beta, self._eps, self._y,
                                       self._mean, self._invstd, self._ws, self._wn, stream)
        else:
            st = self._lib.bns_forward(ctypes.byref(self._sh), self._x, self._gamma, self._beta, self._eps,
                                       ctypes.byref(self._sp), self._y, self._mean, self._invstd, self._ws, self._wn,
                                       stream)
        if st != OK:
            raise BnsError(st, "bns_forward")

    def backward(self):
        st = self._lib.bns_backward(ctypes.byref(self._sh), self._x, self._dy, self._gamma, self._mean, self._invstd,
                                    ctypes.byref(self._sp), self._dx, self._dgamma, self._dbeta, self._ws, self._wn,
                                    torch.cuda.current_stream().cuda_stream)
        if st != OK:
            raise BnsError(st, "bns_backward")


# ----------------------------------------------------------------------------- Eq. 4 and Appendix D
def workspace_bytes_mixed(x, sampling: Sampling) -> int:
    sh = _shape(x)
    sp = sampling._c(sh)
    n = load().bns_workspace_bytes_mixed(ctypes.byref(sh), ctypes.byref(sp))
    if n == 0:
        raise BnsError(-3, "bns_workspace_bytes_mixed (invalid shape or sampling rule)")
    return int(n)


def forward_mixed(x, gamma, beta, eps, mix, sampling: Sampling, workspace=None, y=None, stats=None):
    """bns_forward_mixed: returns (y, mean, invstd, mean_s, mean_v); yv goes to sampling.yv.  `stats` may
    give the four float32[C] output tensors (mean, invstd, mean_s, mean_v)."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    mean, invstd, mean_s, mean_v = stats if stats is not None else (
        torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(4))
    if workspace is None:
        workspace = torch.empty(workspace_bytes_mixed(x, sampling), dtype=torch.uint8, device=x.device)
    st = load().bns_forward_mixed(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps), float(mix),
                                  ctypes.byref(sp), _like(y, x, "y"), _vec(mean, C), _vec(invstd, C), _vec(mean_s, C),
                                  _vec(mean_v, C), workspace.data_ptr(), workspace.numel(), _stream())
    _check(st, "bns_forward_mixed")
    return y, mean, invstd, mean_s, mean_v


def backward_mixed(x, dy, gamma, mean, invstd, mean_s, mean_v, mix, sampling: Sampling, workspace=None, dx=None,
                   grads=None):
    """bns_backward_mixed: returns (dx, dgamma, dbeta); dxv goes to sampling.dxv."""
    _check_virtual(x, sampling)
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    dx = torch.empty_like(x) if dx is None else dx
    dgamma, dbeta = grads if grads is not None else (
        torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    if workspace is None:
        workspace = torch.empty(workspace_bytes_mixed(x, sampling), dtype=torch.uint8, device=x.device)
    st = load().bns_backward_mixed(ctypes.byref(sh), _dev(x), _dev(dy), _vec(gamma, C), _vec(mean, C), _vec(invstd, C),
                                   _vec(mean_s, C), _vec(mean_v, C), float(mix), ctypes.byref(sp), _like(dx, x, "dx"),
                                   _vec(dgamma, C), _vec(dbeta, C), workspace.data_ptr(), workspace.numel(), _stream())
    _check(st, "bns_backward_mixed")
    return dx, dgamma, dbeta


def update_moving_average(mean, invstd, eps, alpha, first_iteration, mean_ma, var_ma):
    """bns_update_moving_average: Eq. 8 on mean_ma / var_ma, in place."""
    C = mean.numel()
    st = load().bns_update_moving_average(C, _vec(mean, C), _vec(invstd, C), float(eps), float(alpha),
                                          1 if first_iteration else 0, _vec(mean_ma, C), _vec(var_ma, C), _stream())
    _check(st, "bns_update_moving_average")


def inference_forward(x, gamma, beta, eps, mean_ma, var_ma, y=None, workspace=None):
    """bns_inference_forward: Eq. 1 with the recorded moving averages; returns y."""
    sh = _shape(x)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    ws, wp, wn = _workspace(x, Sampling.full(), workspace)
    st = load().bns_inference_forward(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps),
                                      _vec(mean_ma, C), _vec(var_ma, C), _like(y, x, "y"), wp, wn, _stream())
    _check(st, "bns_inference_forward")
    return y


# ----------------------------------------------------------------------------- statistics shared by several GPUs
def sync_local_moments(x, sampling: Optional[Sampling], eps, workspace=None):
    """bns_sync_local_moments: float32 [3, C] = (count, mean, M2) of this rank's sampled set; ``sampling=None``
    means that this rank contributes nothing (a count of zero)."""
    sh = _shape(x)
    moments = torch.empty(3, x.shape[1], dtype=torch.float32, device=x.device)
    if sampling is None:
        _check(load().bns_sync_local_moments(ctypes.byref(sh), _dev(x), None, float(eps), moments.data_ptr(), None, 0,
                                             _stream()), "bns_sync_local_moments")
        return moments
    _check_virtual(x, sampling)
    sp = sampling._c(sh)
    ws, wp, wn = _workspace(x, sampling, workspace)
    _check(load().bns_sync_local_moments(ctypes.byref(sh), _dev(x), ctypes.byref(sp), float(eps), moments.data_ptr(),
                                         wp, wn, _stream()), "bns_sync_local_moments")
    return moments


def sync_merge_moments(gathered, eps):
    """bns_sync_merge_moments on a [ranks, 3, C] tensor (an all-gather result): returns (mean, invstd, count),
    count being the sampled points per channel over all ranks (it stays on the device)."""
    R, three, C = gathered.shape
    assert three == 3 and gathered.dtype == torch.float32
    mean, invstd, count = (torch.empty(C, dtype=torch.float32, device=gathered.device) for _ in range(3))
    _check(load().bns_sync_merge_moments(C, R, _dev(gathered), float(eps), mean.data_ptr(), invstd.data_ptr(),
                                         count.data_ptr(), _stream()), "bns_sync_merge_moments")
    return mean, invstd, count


def sync_normalize(x, gamma, beta, mean, invstd, y=None):
    sh = _shape(x)
    C = x.shape[1]
    y = torch.empty_like(x) if y is None else y
    _check(load().bns_sync_normalize(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), _vec(mean, C),
                                     _vec(invstd, C), _like(y, x, "y"), _stream()), "bns_sync_normalize")
    return y


def sync_backward_sums(x, dy, gamma, mean, invstd, dx=None, workspace=None, virtual_rows: Optional[Sampling] = None):
    """bns_sync_backward_sums: returns (dx without the statistics terms, sums float32 [2, C]).  ``virtual_rows``
    is the VIRTUAL rule of the rank that fed virtual samples into the statistics: with dyv set, their gradient
    joins this rank's sums."""
    sh = _shape(x)
    C = x.shape[1]
    dx = torch.empty_like(x) if dx is None else dx
    sums = torch.empty(2, C, dtype=torch.float32, device=x.device)
    rule = virtual_rows if (virtual_rows is not None and virtual_rows.dyv is not None) else Sampling.full()
    ws, wp, wn = _workspace(x, rule, workspace)
    vp = None
    if virtual_rows is not None:
        _check_virtual(x, virtual_rows)
        vr = virtual_rows._c(sh)
        vp = ctypes.byref(vr)
    _check(load().bns_sync_backward_sums(ctypes.byref(sh), _dev(x), _dev(dy), _vec(gamma, C), _vec(mean, C),
                                         _vec(invstd, C), vp, _dev(dx), sums.data_ptr(), wp, wn, _stream()),
           "bns_sync_backward_sums")
    return dx, sums


def sync_backward_apply(x, dy, gamma, mean, invstd, sampling: Optional[Sampling], sums, count, dx, workspace=None):
    """bns_sync_backward_apply: adds the statistics terms to dx on this rank's sampled elements (for a VIRTUAL
    rule: writes dxv).  ``count`` is the merged count from sync_merge_moments; ``sampling=None``: nothing to do."""
    sh = _shape(x)
    C = x.shape[1]
    if sampling is None:
        return dx
    _check_virtual(x, sampling)
    sp = sampling._c(sh)
    ws, wp, wn = _workspace(x, sampling, workspace)
    _check(load().bns_sync_backward_apply(ctypes.byref(sh), _dev(x), _dev(dy), _vec(gamma, C), _vec(mean, C),
                                          _vec(invstd, C), ctypes.byref(sp), _dev(sums), _vec(count, C), _dev(dx),
                                          wp, wn, _stream()), "bns_sync_backward_apply")
    return dx


# ----------------------------------------------------------------------------- BN + residual add + ReLU
def forward_relu(x, residual, gamma, beta, eps, sampling: Sampling, workspace=None):
    """bns_forward_relu: returns (y, mean, invstd) with y = max(0, BN(x) + residual); residual may be None."""
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    y = torch.empty_like(x)
    mean, invstd = (torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    ws, wp, wn = _workspace(x, sampling, workspace)
    st = load().bns_forward_relu(ctypes.byref(sh), _dev(x), None if residual is None else _dev(residual), _vec(gamma, C),
                                 _vec(beta, C), float(eps), ctypes.byref(sp), _dev(y), _vec(mean, C), _vec(invstd, C),
                                 wp, wn, _stream())
    _check(st, "bns_forward_relu")
    return y, mean, invstd


def backward_relu(x, residual, dy, gamma, beta, mean, invstd, sampling: Sampling, workspace=None):
    """bns_backward_relu: returns (dx, dresidual or None, dgamma, dbeta)."""
    sh = _shape(x)
    sp = sampling._c(sh)
    C = x.shape[1]
    dx = torch.empty_like(x)
    dres = None if residual is None else torch.empty_like(x)
    dgamma, dbeta = (torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    ws, wp, wn = _workspace(x, sampling, workspace)
    st = load().bns_backward_relu(ctypes.byref(sh), _dev(x), None if residual is None else _dev(residual), _dev(dy),
                                  _vec(gamma, C), _vec(beta, C), _vec(mean, C), _vec(invstd, C), ctypes.byref(sp),
                                  _dev(dx), None if dres is None else _dev(dres), _vec(dgamma, C), _vec(dbeta, C), wp, wn,
                                  _stream())
    _check(st, "bns_backward_relu")
    return dx, dres, dgamma, dbeta


# ----------------------------------------------------------------------------- channels-last tensors
def _shape_nhwc(x: torch.Tensor) -> _Shape:
    if x.dim() != 4:
        raise TypeError("expected an NHWC tensor")
    N, H, W, C = x.shape
    return _Shape(N, C, H, W, _dtype_code(x))


def forward_nhwc(x, gamma, beta, eps, sampling: Sampling, workspace=None):
    """bns_forward_nhwc on a dense [N,H,W,C] tensor (virtual tensors in `sampling` are [nv,H,W,C] too);
    returns (y, mean, invstd, workspace) - pass the workspace on to backward_nhwc."""
    _check_virtual(x, sampling)
    sh = _shape_nhwc(x)
    sp = sampling._c(sh)
    C = x.shape[3]
    n = load().bns_workspace_bytes_nhwc(ctypes.byref(sh), ctypes.byref(sp))
    if n == 0:
        raise BnsError(-3, "bns_workspace_bytes_nhwc (invalid shape or sampling rule)")
    if workspace is None:
        workspace = torch.empty(int(n), dtype=torch.uint8, device=x.device)
    y = torch.empty_like(x)
    mean, invstd = (torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    st = load().bns_forward_nhwc(ctypes.byref(sh), _dev(x), _vec(gamma, C), _vec(beta, C), float(eps), ctypes.byref(sp),
                                 _dev(y), _vec(mean, C), _vec(invstd, C), workspace.data_ptr(), workspace.numel(),
                                 _stream())
    _check(st, "bns_forward_nhwc")
    return y, mean, invstd, workspace


def backward_nhwc(x, dy, gamma, mean, invstd, sampling: Sampling, workspace):
    """bns_backward_nhwc: returns (dx, dgamma, dbeta)."""
    _check_virtual(x, sampling)
    sh = _shape_nhwc(x)
    sp = sampling._c(sh)
    C = x.shape[3]
    dx = torch.empty_like(x)
    dgamma, dbeta = (torch.empty(C, dtype=torch.float32, device=x.device) for _ in range(2))
    st = load().bns_backward_nhwc(ctypes.byref(sh), _dev(x), _dev(dy), _vec(gamma, C), _vec(mean, C), _vec(invstd, C),
                                  ctypes.byref(sp), _dev(dx), _vec(dgamma, C), _vec(dbeta, C), workspace.data_ptr(),
                                  workspace.numel(), _stream())
    _check(st, "bns_backward_nhwc")
    return dx, dgamma, dbeta


# ----------------------------------------------------------------------------- host-buffer step
def host_arena_bytes(shape, dtype, sampling: Sampling) -> int:
    N, C, H, W = shape
    sh = _Shape(N, C, H, W, F32 if dtype == torch.float32 else BF16)
    sp = sampling._c(sh)
    return int(load().bns_host_arena_bytes(ctypes.byref(sh), ctypes.byref(sp)))


def forward_backward_host(x, dy, gamma, beta, eps, sampling: Sampling, y, dx, mean, invstd, dgamma, dbeta, arena):
    """bns_forward_backward_host: every tensor argument is a (preferably pinned) HOST tensor except
    ``arena`` (CUDA uint8 scratch of ``host_arena_bytes``).  Enqueues copies and kernels on the
    current stream; synchronise before reading the outputs."""
    for t in (x, dy, gamma, beta, y, dx, mean, invstd, dgamma, dbeta):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError("forward_backward_host takes contiguous host tensors")
    N, C, H, W = x.shape
    sh = _Shape(N, C, H, W, _dtype_code(x))
    sp = sampling._c()
    st = load().bns_forward_backward_host(ctypes.byref(sh), x.data_ptr(), dy.data_ptr(), gamma.data_ptr(),
                                          beta.data_ptr(), float(eps), ctypes.byref(sp), y.data_ptr(), dx.data_ptr(),
                                          mean.data_ptr(), invstd.data_ptr(), dgamma.data_ptr(), dbeta.data_ptr(),
                                          arena.data_ptr(), arena.numel(), _stream())
    _check(st, "bns_forward_backward_host")


# ----------------------------------------------------------------------------- measurement hooks
def launch_count() -> int:
    return int(load().bns_launch_count())


def launch_count_reset() -> None:
    load().bns_launch_count_reset()


def profile_enable(on: bool) -> None:
    load().bns_profile_enable(1 if on else 0)


def profile_read(kind: int):
    """(launches, total device milliseconds) of one kernel kind since profiling was enabled."""
    n, ms = ctypes.c_int(0), ctypes.c_float(0.0)
    _check(load().bns_profile_read(int(kind), ctypes.byref(n), ctypes.byref(ms)), "bns_profile_read")
    return int(n.value), float(ms.value)


def set_tuning(name: str, value: int) -> None:
    """bns_set_tuning: launch-shape knobs (see include/bns.h)."""
    _check(load().bns_set_tuning(name.encode(), int(value)), f"bns_set_tuning({name})")


def slab_plan(x: torch.Tensor, sampling: Sampling, backward: bool = False):
    """bns_slab_plan: None when the streaming path serves this shape and rule, else a dict describing the
    one-launch path (channels and blocks per cluster, samples and shared-memory bytes per block, grid)."""
    sh = _shape(x)
    sp = sampling._c(sh)
    out = (ctypes.c_int32 * 6)()
    if not load().bns_slab_plan(ctypes.byref(sh), ctypes.byref(sp), 1 if backward else 0, out):
        return None
    return dict(zip(("channels", "cluster", "rows", "smem_bytes", "grid", "row_lanes"), (int(v) for v in out)))


def wait_timeouts() -> int:
    """bns_wait_timeouts: bounded waits that ran out on this device since the library was loaded."""
    n = ctypes.c_uint32(0)
    _check(load().bns_wait_timeouts(ctypes.byref(n), _stream()), "bns_wait_timeouts")
    return int(n.value)


def kernel_name(kind: int) -> str:
    return load().bns_kernel_name(int(kind)).decode()
