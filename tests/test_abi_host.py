"""CPU-side checks of the C ABI: the library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1810_10962_b200 import bns

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bns.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bns_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = bns.load()
    names = declared_symbols()
    assert {"bns_forward", "bns_backward", "bns_full_bn", "bns_workspace_bytes"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(bns.EXPORTS)


def test_status_strings():
    assert bns.status_string(0) == "ok"
    for code in range(-8, 0):
        assert bns.status_string(code) not in ("ok", "unknown status")


def _call_forward(shape, sp, x=0x1000, gamma=0x2000, beta=0x3000, y=0x4000, mean=0x5000, invstd=0x6000, eps=1e-5,
                  ws=0x10000, ws_bytes=1 << 30):
    """Fake, never dereferenced device addresses: every case below must be refused on the host.  Run only
    where no GPU is visible, so that a check that stopped working cannot send a kernel to a wild address."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("fake device addresses are only used where no GPU can be reached")
    lib = bns.load()
    sh = bns._Shape(*shape)
    return lib.bns_forward(ctypes.byref(sh), x, gamma, beta, eps, ctypes.byref(sp), y, mean, invstd, ws, ws_bytes, None)


def test_forward_rejects_bad_arguments_before_launching():
    idx = np.array([0, 1], np.int32)
    ok = bns.Sampling.batch(idx)._c()
    shape = (8, 16, 8, 8, bns.F32)
    assert _call_forward((0, 16, 8, 8, 0), ok) == -2                       # N = 0
    assert _call_forward((8, 16, 8, 8, 7), ok) == -5                       # dtype
    assert _call_forward((8, 1 << 15, 1 << 10, 1 << 10, 0), ok) == -2      # C*H*W overflows 31 bits
    assert _call_forward(shape, ok, x=0) == -1                             # null x
    assert _call_forward(shape, ok, x=0x1004) == -6                        # misaligned x
    assert _call_forward(shape, ok, eps=0.0) == -2
    assert _call_forward(shape, ok, ws=0) == -7
    assert _call_forward(shape, ok, ws=0x10010) == -7                      # workspace not 256-aligned
    assert _call_forward(shape, ok, ws_bytes=16) == -7
    for bad in ([0, 0], [0, 8], [-1, 2]):                                  # repeated / out of range
        sp = bns.Sampling.batch(np.array(bad, np.int32))._c()
        assert _call_forward(shape, sp) == -4
    sp = bns.Sampling.batch(np.arange(9, dtype=np.int32))._c()             # k > N
    assert _call_forward(shape, sp) == -3
    sp = bns.Sampling.feature(9, 2, np.array([0, 0]))._c()                 # patch taller than the map
    assert _call_forward(shape, sp) == -3
    sp = bns.Sampling.feature(3, 3, np.array([6, 0]))._c()                 # patch leaves the map
    assert _call_forward(shape, sp) == -4
    sp = bns.Sampling.feature(3, 3, np.array([0, -1]))._c()
    assert _call_forward(shape, sp) == -4
    sp = bns._Sampling()
    sp.rule = 9
    assert _call_forward(shape, sp) == -3
    sp = bns._Sampling()
    sp.rule, sp.nv = bns.RULE_VIRTUAL, 0
    assert _call_forward(shape, sp) == -3
    sp.nv = 2                                                              # xv missing
    assert _call_forward(shape, sp) == -1


def test_workspace_bytes_is_zero_for_invalid_and_stable_for_valid():
    lib = bns.load()
    sh = bns._Shape(256, 64, 56, 56, bns.F32)
    sp = bns.Sampling.batch(np.arange(32, dtype=np.int32))._c()
    a = lib.bns_workspace_bytes(ctypes.byref(sh), ctypes.byref(sp))
    assert a > 0 and a == lib.bns_workspace_bytes(ctypes.byref(sh), ctypes.byref(sp)) and a % 256 == 0
    bad = bns._Shape(256, 64, 56, -1, bns.F32)
    assert lib.bns_workspace_bytes(ctypes.byref(bad), ctypes.byref(sp)) == 0


def test_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros(2, 3, 4, 4)
    with pytest.raises(TypeError):
        bns.forward(x, torch.ones(3), torch.zeros(3), 1e-5, bns.Sampling.full(),
                    workspace=torch.empty(1 << 20, dtype=torch.uint8))


def test_binding_checks_the_length_of_device_offsets():
    """Per-sample / per-map patch offsets are indexed by sample (and channel) on the device, so the binding
    refuses a tensor that does not hold one pair for each.  (Checked before anything touches the tensor's
    memory, so an object standing in for a CUDA tensor serves on a machine without a GPU.)"""
    import torch

    class FakeCudaInt32(torch.Tensor):
        is_cuda = True

    def offsets(pairs):
        return torch.zeros(pairs, 2, dtype=torch.int32).as_subclass(FakeCudaInt32)

    shape = bns._Shape(8, 16, 8, 8, bns.F32)
    bns.Sampling.feature(2, 2, offsets(8), bns.OFF_PER_SAMPLE)._c(shape)
    bns.Sampling.feature(2, 2, offsets(8 * 16), bns.OFF_PER_MAP)._c(shape)
    for mode, pairs in ((bns.OFF_PER_SAMPLE, 7), (bns.OFF_PER_SAMPLE, 8 * 16), (bns.OFF_PER_MAP, 8), (bns.OFF_PER_MAP, 127)):
        with pytest.raises(TypeError):
            bns.Sampling.feature(2, 2, offsets(pairs), mode)._c(shape)


def _plan(N, C, H, W, dtype, sampling, backward):
    lib = bns.load()
    sh = bns._Shape(N, C, H, W, dtype)
    sp = sampling._c(sh)
    out = (ctypes.c_int32 * 6)()
    ok = lib.bns_slab_plan(ctypes.byref(sh), ctypes.byref(sp), 1 if backward else 0, out)
    return dict(zip(("channels", "cluster", "rows", "smem_bytes", "grid", "row_lanes"), out)) if ok else None


def test_onchip_plans_respect_the_hardware_limits():
    """Host logic of the one-launch path: which layers take it by default, and that every plan it makes fits
    a thread-block cluster (at most 8 blocks, at most 227 KB of shared memory each, row segments of whole
    16-byte units, every sample held by exactly one block)."""
    full = bns.Sampling.full()
    try:
        # defaults: small tensors only, and not for small sampled sets
        assert _plan(128, 32, 16, 16, bns.F32, full, False) is not None                    # 4 MiB
        assert _plan(256, 256, 14, 14, bns.BF16, full, False) is None                      # 24.5 MiB
        assert _plan(128, 32, 16, 16, bns.F32, bns.Sampling.feature(4, 4, np.array([0, 0])), True) is None
        assert _plan(8, 16, 8, 8, bns.F32, bns.Sampling.batch(np.array([1, 5], np.int32)), False) is None
        bns.set_tuning("slab_max_mb", 1 << 20)
        bns.set_tuning("slab_small_sets", 1)
        rng = np.random.default_rng(5)
        seen = 0
        for _ in range(400):
            N, C = int(rng.integers(1, 300)), int(rng.integers(1, 40)) * int(rng.choice([1, 2, 8, 16]))
            H, W = int(rng.integers(1, 40)), int(rng.integers(1, 40))
            dtype = int(rng.integers(0, 2))
            eb = 4 if dtype == bns.F32 else 2
            for backward in (False, True):
                p = _plan(N, C, H, W, dtype, full, backward)
                if p is None:
                    continue
                seen += 1
                G, R = p["channels"], p["cluster"]
                assert 1 <= R <= 8 and R <= N and p["smem_bytes"] <= 227 * 1024
                assert C % G == 0 and (G * H * W * eb) % 16 == 0 and G * H * W * eb // 16 <= 256
                assert p["rows"] == -(-N // R) and p["grid"] == (C // G) * R
                assert p["smem_bytes"] >= (2 if backward else 1) * p["rows"] * G * H * W * eb
        assert seen > 50
        # a channel whose samples cannot fit eight blocks' shared memory keeps streaming
        assert _plan(256, 64, 56, 56, bns.F32, full, True) is None
    finally:
        bns.set_tuning("slab_max_mb", 6)
        bns.set_tuning("slab_small_sets", 0)
