"""ctypes front end of the double-precision CPU oracle (``bns_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg.  It has no dependency on the CUDA library and the CUDA library has none on it.

All tensors are numpy arrays in NCHW.  Activations and gradients are passed as float32 (bf16 data
is widened exactly before the call); every result is float64.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

from .build import build as _build

RULE_FULL, RULE_BATCH, RULE_FEATURE, RULE_VIRTUAL = 0, 1, 2, 3
OFFSETS_SHARED, OFFSETS_PER_SAMPLE, OFFSETS_PER_MAP = 0, 1, 2


class _CSampling(ctypes.Structure):
    _fields_ = [
        ("rule", ctypes.c_int),
        ("k", ctypes.c_int),
        ("sample_idx", ctypes.c_void_p),
        ("ph", ctypes.c_int),
        ("pw", ctypes.c_int),
        ("offset_mode", ctypes.c_int),
        ("offsets", ctypes.c_void_p),
        ("nv", ctypes.c_int),
    ]


@dataclass
class Sampling:
    """Which elements enter the statistics (Eq. 3): the paper's S."""
    rule: int = RULE_FULL
    sample_idx: Optional[np.ndarray] = None   # BATCH: int32 [k]
    ph: int = 0                               # FEATURE
    pw: int = 0
    offset_mode: int = OFFSETS_SHARED
    offsets: Optional[np.ndarray] = None      # FEATURE: int32 [1|N|N*C, 2]
    nv: int = 0                               # VIRTUAL

    @staticmethod
    def full():
        return Sampling(RULE_FULL)

    @staticmethod
    def batch(sample_idx):
        return Sampling(RULE_BATCH, sample_idx=np.ascontiguousarray(sample_idx, dtype=np.int32))

    @staticmethod
    def feature(ph, pw, offsets, offset_mode=OFFSETS_SHARED):
        off = np.ascontiguousarray(offsets, dtype=np.int32).reshape(-1, 2)
        return Sampling(RULE_FEATURE, ph=int(ph), pw=int(pw), offset_mode=int(offset_mode), offsets=off)

    @staticmethod
    def virtual(nv):
        return Sampling(RULE_VIRTUAL, nv=int(nv))

    def _c(self):
        keep = []
        c = _CSampling()
        c.rule = self.rule
        if self.rule == RULE_BATCH:
            idx = np.ascontiguousarray(self.sample_idx, dtype=np.int32)
            keep.append(idx)
            c.k = idx.size
            c.sample_idx = idx.ctypes.data
        if self.rule == RULE_FEATURE:
            off = np.ascontiguousarray(self.offsets, dtype=np.int32)
            keep.append(off)
            c.ph, c.pw, c.offset_mode = self.ph, self.pw, self.offset_mode
            c.offsets = off.ctypes.data
        c.nv = self.nv
        return c, keep


_lib = None


def _library():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build())
        lib.oracle_sample_count.restype = ctypes.c_longlong
        lib.oracle_adder_tree_depth_ratio.restype = ctypes.c_double
        lib.oracle_forward.restype = None
        lib.oracle_backward.restype = None
        lib.oracle_selection_mask.restype = None
        lib.oracle_forward_mixed.restype = None
        lib.oracle_backward_mixed.restype = None
        lib.oracle_moving_average.restype = None
        lib.oracle_inference_forward.restype = None
        _lib = lib
    return _lib


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a):
    return ctypes.c_void_p(None if a is None else a.ctypes.data)


def _channels(channels, C):
    if channels is None:
        return None, C
    ch = np.ascontiguousarray(channels, dtype=np.int32)
    assert ch.ndim == 1 and ch.size > 0 and ch.min() >= 0 and ch.max() < C
    return ch, int(ch.size)


def _check_offsets(sp: Sampling, N, C, H, W):
    if sp.rule == RULE_BATCH:
        idx = sp.sample_idx
        assert idx.size >= 1 and idx.min() >= 0 and idx.max() < N and np.unique(idx).size == idx.size
    if sp.rule == RULE_FEATURE:
        count = {OFFSETS_SHARED: 1, OFFSETS_PER_SAMPLE: N, OFFSETS_PER_MAP: N * C}[sp.offset_mode]
        off = sp.offsets
        assert off.shape == (count, 2)
        assert 1 <= sp.ph <= H and 1 <= sp.pw <= W
        assert off[:, 0].min() >= 0 and off[:, 0].max() <= H - sp.ph
        assert off[:, 1].min() >= 0 and off[:, 1].max() <= W - sp.pw
    if sp.rule == RULE_VIRTUAL:
        assert sp.nv >= 1


def threads() -> int:
    """Host threads the oracle's channel loop uses."""
    return int(_library().oracle_threads())


def sample_count(N, H, W, sp: Sampling) -> int:
    c, _keep = sp._c()
    return int(_library().oracle_sample_count(N, H, W, ctypes.byref(c)))


def adder_tree_depth_ratio(N, H, W, sp: Sampling) -> float:
    c, _keep = sp._c()
    return float(_library().oracle_adder_tree_depth_ratio(N, H, W, ctypes.byref(c)))


def selection_mask(N, C, H, W, sp: Sampling) -> np.ndarray:
    _check_offsets(sp, N, C, H, W)
    c, _keep = sp._c()
    mask = np.zeros((N, C, H, W), dtype=np.uint8)
    _library().oracle_selection_mask(N, C, H, W, ctypes.byref(c), _ptr(mask))
    return mask


@dataclass
class Forward:
    y: Optional[np.ndarray]
    yv: Optional[np.ndarray]
    mean: np.ndarray
    var: np.ndarray
    invstd: np.ndarray


@dataclass
class Backward:
    dx: Optional[np.ndarray]
    dxv: Optional[np.ndarray]
    dgamma: np.ndarray
    dbeta: np.ndarray


def forward(x, gamma, beta, eps, sp: Sampling, xv=None, channels: Optional[Sequence[int]] = None,
            want_y=True, want_yv=True) -> Forward:
    """Eq. 1 with the statistics of Eq. 3 (Eq. 2 for the FULL rule), for the listed channels."""
    x = _f32(x)
    N, C, H, W = x.shape
    _check_offsets(sp, N, C, H, W)
    xv = _f32(xv)
    if sp.rule == RULE_VIRTUAL:
        assert xv is not None and xv.shape == (sp.nv, C, H, W)
    gamma, beta = _f32(gamma), _f32(beta)
    assert gamma.shape == (C,) and beta.shape == (C,) and eps > 0
    ch, nch = _channels(channels, C)
    y = np.empty((N, nch, H, W), dtype=np.float64) if want_y else None
    yv = np.empty((sp.nv, nch, H, W), dtype=np.float64) if (sp.rule == RULE_VIRTUAL and want_yv) else None
    mean, var, invstd = (np.empty(nch, dtype=np.float64) for _ in range(3))
    c, _keep = sp._c()
    _library().oracle_forward(N, C, H, W, _ptr(x), _ptr(xv), _ptr(gamma), _ptr(beta), ctypes.c_double(eps),
                              ctypes.byref(c), _ptr(ch), nch, _ptr(y), _ptr(yv), _ptr(mean), _ptr(var),
                              _ptr(invstd))
    return Forward(y, yv, mean, var, invstd)


def backward(x, dy, gamma, mean, var, eps, sp: Sampling, xv=None, dyv=None,
             channels: Optional[Sequence[int]] = None, want_dx=True, want_dxv=True) -> Backward:
    """Eq. 5 / Eq. 6 for the listed channels; ``mean`` and ``var`` are ``forward``'s for those channels."""
    x, dy = _f32(x), _f32(dy)
    N, C, H, W = x.shape
    assert dy.shape == x.shape
    _check_offsets(sp, N, C, H, W)
    xv, dyv = _f32(xv), _f32(dyv)
    if sp.rule == RULE_VIRTUAL:
        assert xv is not None and xv.shape == (sp.nv, C, H, W)
        assert dyv is None or dyv.shape == xv.shape
    gamma = _f32(gamma)
    ch, nch = _channels(channels, C)
    mean = np.ascontiguousarray(mean, dtype=np.float64)
    var = np.ascontiguousarray(var, dtype=np.float64)
    assert mean.shape == (nch,) and var.shape == (nch,)
    dx = np.empty((N, nch, H, W), dtype=np.float64) if want_dx else None
    dxv = np.empty((sp.nv, nch, H, W), dtype=np.float64) if (sp.rule == RULE_VIRTUAL and want_dxv) else None
    dgamma, dbeta = (np.empty(nch, dtype=np.float64) for _ in range(2))
    c, _keep = sp._c()
    _library().oracle_backward(N, C, H, W, _ptr(x), _ptr(xv), _ptr(dy), _ptr(dyv), _ptr(gamma), _ptr(mean),
                               _ptr(var), ctypes.c_double(eps), ctypes.byref(c), _ptr(ch), nch, _ptr(dx),
                               _ptr(dxv), _ptr(dgamma), _ptr(dbeta))
    return Backward(dx, dxv, dgamma, dbeta)


# ----------------------------------------------------------------------------- Eq. 4: VDN combined with a sampling rule
@dataclass
class ForwardMixed:
    y: Optional[np.ndarray]
    yv: Optional[np.ndarray]
    mean: np.ndarray
    var: np.ndarray
    invstd: np.ndarray
    mean_s: np.ndarray
    var_s: np.ndarray
    mean_v: np.ndarray
    var_v: np.ndarray


def forward_mixed(x, xv, gamma, beta, eps, mix, sp: Sampling, channels=None, want_y=True, want_yv=True) -> ForwardMixed:
    """Eq. 4: E = mix*E[xv] + (1-mix)*E[x_s], Var likewise; Eq. 1 on x and xv with the mixed statistics."""
    x, xv = _f32(x), _f32(xv)
    N, C, H, W = x.shape
    assert sp.rule in (RULE_BATCH, RULE_FEATURE) and xv.shape[1:] == (C, H, W)
    _check_offsets(sp, N, C, H, W)
    nv = xv.shape[0]
    gamma, beta = _f32(gamma), _f32(beta)
    ch, nch = _channels(channels, C)
    y = np.empty((N, nch, H, W), dtype=np.float64) if want_y else None
    yv = np.empty((nv, nch, H, W), dtype=np.float64) if want_yv else None
    vec = [np.empty(nch, dtype=np.float64) for _ in range(6)]
    c, _keep = sp._c()
    _library().oracle_forward_mixed(N, C, H, W, _ptr(x), _ptr(xv), nv, _ptr(gamma), _ptr(beta), ctypes.c_double(eps),
                                    ctypes.c_double(mix), ctypes.byref(c), _ptr(ch), nch, _ptr(y), _ptr(yv),
                                    *[_ptr(v) for v in vec])
    mean, var, mean_s, var_s, mean_v, var_v = vec
    return ForwardMixed(y, yv, mean, var, 1.0 / np.sqrt(var + eps), mean_s, var_s, mean_v, var_v)


def backward_mixed(x, xv, dy, dyv, gamma, fwd: ForwardMixed, eps, mix, sp: Sampling, channels=None) -> Backward:
    """Chain rule through Eq. 4 (see bns_oracle.c); `fwd` is forward_mixed's result for the same channels."""
    x, xv, dy, dyv = _f32(x), _f32(xv), _f32(dy), _f32(dyv)
    N, C, H, W = x.shape
    nv = xv.shape[0]
    gamma = _f32(gamma)
    ch, nch = _channels(channels, C)
    dx = np.empty((N, nch, H, W), dtype=np.float64)
    dxv = np.empty((nv, nch, H, W), dtype=np.float64)
    dgamma, dbeta = (np.empty(nch, dtype=np.float64) for _ in range(2))
    c, _keep = sp._c()
    _library().oracle_backward_mixed(N, C, H, W, _ptr(x), _ptr(xv), nv, _ptr(dy), _ptr(dyv), _ptr(gamma),
                                     _ptr(fwd.mean), _ptr(fwd.var), _ptr(fwd.mean_s), _ptr(fwd.mean_v),
                                     ctypes.c_double(eps), ctypes.c_double(mix), ctypes.byref(c), _ptr(ch), nch,
                                     _ptr(dx), _ptr(dxv), _ptr(dgamma), _ptr(dbeta))
    return Backward(dx, dxv, dgamma, dbeta)


# ----------------------------------------------------------------------------- Appendix D: moving average, validation forward
def moving_average(X, X_ma, alpha, first_iteration) -> np.ndarray:
    """Eq. 8: returns the updated moving average (X_ma is not modified)."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    out = np.array(X_ma, dtype=np.float64, copy=True) if X_ma is not None else np.zeros_like(X)
    _library().oracle_moving_average(X.size, int(bool(first_iteration)), ctypes.c_double(alpha), _ptr(X), _ptr(out))
    return out


def inference_forward(x, gamma, beta, eps, E_ma, Var_ma) -> np.ndarray:
    """Eq. 1 with the recorded moving averages in place of the batch statistics."""
    x = _f32(x)
    N, C, H, W = x.shape
    gamma, beta = _f32(gamma), _f32(beta)
    E_ma = np.ascontiguousarray(E_ma, dtype=np.float64)
    Var_ma = np.ascontiguousarray(Var_ma, dtype=np.float64)
    y = np.empty(x.shape, dtype=np.float64)
    _library().oracle_inference_forward(N, C, H, W, _ptr(x), _ptr(gamma), _ptr(beta), ctypes.c_double(eps), _ptr(E_ma),
                                        _ptr(Var_ma), _ptr(y))
    return y


# ----------------------------------------------------------------------------- BN followed by a residual add and ReLU
# Not an equation of the paper: the step that follows every BN layer of the ResNets it trains
# (y = max(0, BN(x) + r)).  Stated here by composing the pinned BN forward/backward above with the
# definition of the rectifier, so that a fused GPU version has something to be compared with.
@dataclass
class ForwardAct:
    y: np.ndarray        # max(0, z)
    z: np.ndarray        # BN(x) + residual, before the rectifier
    mean: np.ndarray
    var: np.ndarray
    invstd: np.ndarray


def forward_relu(x, residual, gamma, beta, eps, sp: Sampling, channels=None) -> ForwardAct:
    assert sp.rule != RULE_VIRTUAL
    f = forward(x, gamma, beta, eps, sp, channels=channels)
    z = f.y
    if residual is not None:
        r = _f32(residual).astype(np.float64)
        z = z + (r if channels is None else r[:, np.asarray(channels)])
    return ForwardAct(np.maximum(z, 0.0), z, f.mean, f.var, f.invstd)


def backward_relu(x, dy, gamma, fwd: ForwardAct, eps, sp: Sampling, channels=None):
    """Returns (Backward for the BN part with the rectifier's gradient applied, dresidual = dy * [z > 0])."""
    dyf = _f32(dy)
    sel = slice(None) if channels is None else np.asarray(channels)
    g_sel = np.where(fwd.z > 0.0, dyf[:, sel].astype(np.float64), 0.0)
    # the C oracle takes float32 gradients: g is dy or 0, both exactly representable
    g = np.zeros_like(dyf)
    g[:, sel] = g_sel.astype(np.float32)
    b = backward(x, g, gamma, fwd.mean, fwd.var, eps, sp, channels=channels)
    return b, g_sel
