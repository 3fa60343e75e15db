#!/usr/bin/env python
"""Benchmark of the sampled-BN forward+backward path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A *step* is one forward+backward of every layer of the workload through the C ABI.  The K steps of
``--steps`` are timed as one loop between two CUDA events; that loop is repeated (at least 30 times and for
at least ``--seconds``) and the reported time per step is the median over the repetitions, with the
minimum beside it.  The default
workload is the ImageNet ResNet-18 stage-1 layer, fp32 (256,64,56,56), once with Batch Sampling
(k = 32 of 256) and once with Feature Sampling (8x8 patch), and the same layer through the library's
full BN for the speed-up figure.  The metric is algorithmic GB/s: the bytes the method itself must
move, (2+r)Eb forward and (3+3r)Eb backward for a sampled layer with sampling ratio r (8Eb for full
BN), divided by device time.  One JSON line is printed by rank 0.

With N > 1 (launched by torchrun) every rank runs the same layers on its own GPU: BN statistics are
local to a GPU in the paper (Sec. 5, "Experimental Setup"), so the path has no exchange step and the
ranks are independent replicas; the value is the bytes of all ranks over the slowest rank's time.

``--impl reference`` times the double-precision CPU oracle, as it stands, on a bounded sample
(a subset of channels, which are independent units of work) of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bns_inputs as I  # noqa: E402

EPS = 1e-5
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of backward pass 1 (fp32, 16-byte vectors, writing dx)
# on the default workload's layer shape (256x64x56x56 fp32), from an ncu capture of this very kernel; reported
# only for that workload.  None whenever the kernel has changed since the counters were taken.
BWD_REDUCE_DRAM_TRAFFIC_BYTES = 577_856_512   # 411.11 MB read + 164.92 MB written (rest of dx still dirty in L2)


# ----------------------------------------------------------------------------- workloads
class Layer:
    """One BN layer of a workload: shape, element type, sampling rule and how often it occurs."""

    def __init__(self, name, N, C, H, W, dtype, rule, count=1, **kw):
        self.name, self.N, self.C, self.H, self.W = name, N, C, H, W
        self.dtype, self.rule, self.count, self.kw = dtype, rule, count, kw

    @property
    def elems(self):
        return self.N * self.C * self.H * self.W

    @property
    def ebytes(self):
        return 4 if self.dtype == "f32" else 2

    def sampled_per_channel(self):
        m = self.N * self.H * self.W
        if self.rule == "full":
            return m
        if self.rule == "batch":
            return self.kw["k"] * self.H * self.W
        if self.rule in ("feature", "mixed", "relu"):
            return self.N * self.kw["ph"] * self.kw["pw"]
        return self.kw["nv"] * self.H * self.W

    def algorithmic_bytes(self):
        """Bytes one forward+backward of this layer must move (statistics vectors included)."""
        E, b, C = self.elems, self.ebytes, self.C
        vec = 16 * C
        if self.rule == "full":
            return 8 * E * b + 2 * vec
        if self.rule == "relu":
            # forward reads x, residual, the patches and writes y; backward reads x, residual, dy, writes dx and
            # dresidual; the fix-up reads x, residual, dy on S and writes dx there
            r = self.sampled_per_channel() / (self.N * self.H * self.W)
            return int(round((8 + 5 * r) * E * b)) + 2 * vec
        if self.rule == "mixed":
            ev = self.kw["nv"] * C * self.H * self.W * 4      # xv is fp32: statistics, yv, and dxv as for VDN
            r = self.sampled_per_channel() / (self.N * self.H * self.W)
            return int(round((5 + 4 * r) * E * b)) + 5 * ev + 2 * vec
        if self.rule == "virtual":
            ev = self.kw["nv"] * C * self.H * self.W * 4      # xv is fp32
            # forward: read xv (statistics), read xv + write yv, read x, write y; backward: read x, dy, write dx,
            # read xv, write dxv
            return 5 * E * b + 5 * ev + 2 * vec
        r = self.sampled_per_channel() / (self.N * self.H * self.W)
        return int(round((5 + 4 * r) * E * b)) + 2 * vec


def workload_layers(name):
    if name == "resnet18_stage1":
        shape = dict(N=256, C=64, H=56, W=56, dtype="f32")
        return [Layer("bs32", rule="batch", k=32, **shape), Layer("fs8x8", rule="feature", ph=8, pw=8, **shape)]
    if name == "cifar":
        return [Layer(f"fs4x4_c{C}_h{H}", 128, C, H, H, "f32", "feature", ph=4, pw=4) for C, H in I.cifar_resnet_layers()]
    if name == "vdn":
        return [Layer("vdn2", 256, 128, 28, 28, "bf16", "virtual", nv=2)]
    if name == "resnet50":
        layers, seen = [], {}
        for C, H in I.resnet50_bn_layers():
            seen[(C, H)] = seen.get((C, H), 0) + 1
        for (C, H), cnt in sorted(seen.items(), key=lambda t: (-t[0][1], t[0][0])):
            p = max(1, H // 8)
            layers.append(Layer(f"fs{p}x{p}_c{C}_h{H}", 256, C, H, H, "bf16", "feature", count=cnt, ph=p, pw=p))
        return layers
    if name == "fs_vdn":
        # the paper's most accurate variant (Table 2, "FS+VDN"): Eq. 4 with a patch and two virtual samples
        return [Layer("fs8x8_vdn2", 256, 64, 56, 56, "f32", "mixed", ph=8, pw=8, nv=2, mix=0.5)]
    if name == "fs_relu":
        # the block a ResNet actually runs: BN (Feature Sampling) + residual add + ReLU, fused
        return [Layer("fs8x8_res_relu", 256, 64, 56, 56, "f32", "relu", ph=8, pw=8)]
    if name == "tiny":
        return [Layer("bs2", 8, 16, 8, 8, "f32", "batch", k=2)]
    raise SystemExit(f"unknown workload {name}")


def selected_layers(args):
    layers = workload_layers(args.workload)
    seeds = [layer_seed(args.workload, i) for i in range(len(layers))]
    if args.only:
        keep = set(args.only.split(","))
        pairs = [(l, s) for l, s in zip(layers, seeds) if l.name in keep]
        if not pairs:
            raise SystemExit(f"--only {args.only}: no such layer in {[l.name for l in layers]}")
        layers, seeds = [p[0] for p in pairs], [p[1] for p in pairs]
    return layers, seeds


def layer_seed(workload, index):
    return 1810 + 100 * (["tiny", "cifar", "resnet18_stage1", "vdn", "resnet50", "fs_vdn", "fs_relu"].index(workload) + 1) + index


def host_inputs(layer: Layer, seed):
    """Seeded host inputs of a layer (float32 arrays holding values exact in the layer's dtype)."""
    N, C, H, W = layer.N, layer.C, layer.H, layer.W
    gen = I.tiny_activations if max(H, W) <= 8 and N <= 8 else I.correlated_activations
    x = gen(N, C, H, W, seed)
    dy = I.upstream_gradient(x.shape, seed)
    if layer.dtype == "bf16":
        x, dy = I.round_to_bf16(x), I.round_to_bf16(dy)
    gamma, beta = I.affine_parameters(C, seed)
    extra = {}
    if layer.rule == "batch":
        extra["sample_idx"] = I.batch_sample_indices(N, layer.kw["k"], seed, contiguous=True)
    elif layer.rule == "feature":
        extra["offsets"] = I.patch_offsets(N, C, H, W, layer.kw["ph"], layer.kw["pw"], I.OFFSETS_SHARED, seed)
    elif layer.rule == "virtual":
        extra["xv"] = I.virtual_samples(layer.kw["nv"], C, H, W, seed)
    elif layer.rule == "mixed":
        extra["offsets"] = I.patch_offsets(N, C, H, W, layer.kw["ph"], layer.kw["pw"], I.OFFSETS_SHARED, seed)
        extra["xv"] = I.virtual_samples(layer.kw["nv"], C, H, W, seed)
    elif layer.rule == "relu":
        extra["offsets"] = I.patch_offsets(N, C, H, W, layer.kw["ph"], layer.kw["pw"], I.OFFSETS_SHARED, seed)
        extra["residual"] = I.upstream_gradient(x.shape, seed, I.TAG_XV)
    return dict(x=x, dy=dy, gamma=gamma, beta=beta, **extra)


def device_inputs(layer: Layer, seed, torch):
    """The same recipe as host_inputs, drawn on the device (torch's generator instead of the host one): used for
    the secondary workloads, whose inputs no CPU code reads.  3x3 box blur (replicated border) of N(0,1) noise
    plus a per-channel offset U(-1,1); dy, residual and virtual samples N(0,1); gamma U(0.5,1.5); beta N(0, 0.1)."""
    import torch.nn.functional as F
    N, C, H, W = layer.N, layer.C, layer.H, layer.W
    dt = torch.float32 if layer.dtype == "f32" else torch.bfloat16
    g = torch.Generator(device="cuda")
    g.manual_seed(int(seed))
    offset = torch.rand(C, generator=g, device="cuda") * 2.0 - 1.0
    x = torch.empty(N, C, H, W, device="cuda", dtype=dt)
    block = max(1, (1 << 26) // max(1, C * H * W))           # sample blocks keep the fp32 temporaries small
    for n0 in range(0, N, block):
        n1 = min(N, n0 + block)
        noise = torch.randn(n1 - n0, C, H, W, generator=g, device="cuda")
        blurred = F.avg_pool2d(F.pad(noise, (1, 1, 1, 1), mode="replicate"), 3, stride=1)
        x[n0:n1] = (blurred + offset[None, :, None, None]).to(dt)
    dy = torch.empty(N, C, H, W, device="cuda", dtype=dt)
    for n0 in range(0, N, block):
        n1 = min(N, n0 + block)
        dy[n0:n1] = torch.randn(n1 - n0, C, H, W, generator=g, device="cuda").to(dt)
    out = dict(x=x, dy=dy, gamma=torch.rand(C, generator=g, device="cuda") + 0.5,
               beta=torch.randn(C, generator=g, device="cuda") * 0.1)
    if layer.rule == "batch":
        out["sample_idx"] = I.batch_sample_indices(N, layer.kw["k"], seed, contiguous=True)
    if layer.rule in ("feature", "mixed", "relu"):
        out["offsets"] = I.patch_offsets(N, C, H, W, layer.kw["ph"], layer.kw["pw"], I.OFFSETS_SHARED, seed)
    if layer.rule in ("virtual", "mixed"):
        out["xv"] = torch.randn(layer.kw["nv"], C, H, W, generator=g, device="cuda")
    if layer.rule == "relu":
        out["residual"] = torch.randn(N, C, H, W, generator=g, device="cuda").to(dt)
    return out


# ----------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}
    REJECT = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}

    def __init__(self, index, period=0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        while self.ok and not self._halt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def clocks_rejected(clocks):
    if set(clocks["reasons"]) & ClockSampler.REJECT:
        return True
    if clocks["sm_mhz"] and clocks["sm_max_mhz"] and clocks["sm_mhz"] < 0.6 * clocks["sm_max_mhz"] and not clocks["reasons"]:
        return True     # stuck low with no reason: a leftover clock lock
    return False


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ----------------------------------------------------------------------------- the GPU arm
class DeviceLayer:
    """Device buffers of one layer (several rotating sets of x, dy, y, dx) and its launch closures."""

    def __init__(self, layer: Layer, host, sets, torch, bns, full_bn=False, nhwc=False):
        self.layer, self.bns, self.torch = layer, bns, torch
        self.full = full_bn or layer.rule == "full"
        self.mixed = layer.rule == "mixed" and not self.full
        self.relu = layer.rule == "relu"      # the full-BN comparison runs through the same fused kernels
        self.nhwc = nhwc
        dt = torch.float32 if layer.dtype == "f32" else torch.bfloat16

        def dev(a):
            t = a if torch.is_tensor(a) else torch.from_numpy(a).cuda().to(dt)   # exact: the values are representable in dt
            return t.permute(0, 2, 3, 1).contiguous() if nhwc else t

        def vec(a):
            return a if torch.is_tensor(a) else torch.from_numpy(a).cuda()

        x, dy = dev(host["x"]), dev(host["dy"])
        self.sets = [(x, dy, torch.empty_like(x), torch.empty_like(x))]
        for _ in range(sets - 1):
            self.sets.append((x.clone(), dy.clone(), torch.empty_like(x), torch.empty_like(x)))
        self.gamma, self.beta = vec(host["gamma"]), vec(host["beta"])
        C = layer.C
        self.mean, self.invstd, self.dgamma, self.dbeta = (torch.empty(C, device="cuda") for _ in range(4))
        if nhwc:
            if layer.rule not in ("batch", "feature", "full"):
                raise SystemExit("--layout nhwc is benchmarked for the batch, feature and full rules")
            if self.full:
                self.sp = bns.Sampling.full()
            elif layer.rule == "batch":
                self.sp = bns.Sampling.batch(host["sample_idx"])
            else:
                self.sp = bns.Sampling.feature(layer.kw["ph"], layer.kw["pw"], host["offsets"])
            self.ws = None
            return
        if self.relu:
            self.sp = (bns.Sampling.full() if self.full
                       else bns.Sampling.feature(layer.kw["ph"], layer.kw["pw"], host["offsets"]))
            self.residual = dev(host["residual"])
            self.ws = bns.new_workspace(x, self.sp)
            return
        if self.full:
            self.sp = bns.Sampling.full()
        elif layer.rule == "batch":
            self.sp = bns.Sampling.batch(host["sample_idx"])
        elif layer.rule == "feature":
            self.sp = bns.Sampling.feature(layer.kw["ph"], layer.kw["pw"], host["offsets"])
        elif layer.rule == "mixed":
            xv = vec(host["xv"])
            self.sp = bns.Sampling.feature(layer.kw["ph"], layer.kw["pw"], host["offsets"]).with_virtual(
                xv, yv=torch.empty_like(xv), dyv=None, dxv=torch.empty_like(xv))
            self.mean_s, self.mean_v = (torch.empty(C, device="cuda") for _ in range(2))
            self.ws = torch.empty(bns.workspace_bytes_mixed(x, self.sp), dtype=torch.uint8, device="cuda")
            return
        else:
            xv = vec(host["xv"])
            self.sp = bns.Sampling.virtual(xv, yv=torch.empty_like(xv), dyv=None, dxv=torch.empty_like(xv))
        self.ws = bns.new_workspace(x, self.sp)
        # argument marshalling done once per buffer set; a step is then two C calls per layer
        self.calls = [bns.Prepared(sx, sdy, self.gamma, self.beta, EPS, self.sp, sy, sdx, self.mean, self.invstd,
                                   self.dgamma, self.dbeta, self.ws, full_bn_entry=self.full)
                      for sx, sdy, sy, sdx in self.sets]

    def step(self, i):
        if self.nhwc:
            x, dy, _, _ = self.sets[i % len(self.sets)]
            b = self.bns
            _, mean, invstd, self.ws = b.forward_nhwc(x, self.gamma, self.beta, EPS, self.sp, workspace=self.ws)
            b.backward_nhwc(x, dy, self.gamma, mean, invstd, self.sp, self.ws)
            return
        if self.relu:
            x, dy, _, _ = self.sets[i % len(self.sets)]
            b = self.bns
            _, mean, invstd = b.forward_relu(x, self.residual, self.gamma, self.beta, EPS, self.sp, workspace=self.ws)
            b.backward_relu(x, self.residual, dy, self.gamma, self.beta, mean, invstd, self.sp, workspace=self.ws)
            return
        if self.mixed:
            x, dy, y, dx = self.sets[i % len(self.sets)]
            b, mix = self.bns, self.layer.kw["mix"]
            b.forward_mixed(x, self.gamma, self.beta, EPS, mix, self.sp, workspace=self.ws, y=y,
                            stats=(self.mean, self.invstd, self.mean_s, self.mean_v))
            b.backward_mixed(x, dy, self.gamma, self.mean, self.invstd, self.mean_s, self.mean_v, mix, self.sp,
                             workspace=self.ws, dx=dx, grads=(self.dgamma, self.dbeta))
            return
        call = self.calls[i % len(self.calls)]
        call.forward()
        call.backward()


def capture_steps(torch, step, sets):
    """Captures `sets` consecutive steps (one per rotating buffer set) into a CUDA graph, so that the
    timed loop replays kernels without per-call host work.  Returns None if capture is not possible."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(sets):
                step(i)                      # warm up on the capture stream
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(sets):
                step(i)
        graph.replay()
        torch.cuda.synchronize()
        return graph
    except Exception as exc:                 # keep measuring eagerly
        print(f"bench: CUDA graph capture failed ({exc}); timing eager launches", file=sys.stderr)
        torch.cuda.synchronize()
        return None


class GraphedSteps:
    """Step function for time_steps: a loop of n steps is run as n // sets graph replays (each replay is
    `sets` steps) plus n % sets eager steps, so exactly n steps execute."""

    def __init__(self, graph, step, sets):
        self.graph, self.step, self.sets = graph, step, sets
        self.remaining = self.covered = 0

    def begin(self, n):
        self.remaining, self.covered = n, 0

    def __call__(self, i):
        if self.covered == 0:
            if self.remaining >= self.sets:
                self.graph.replay()
                self.covered = self.sets
            else:
                self.step(i)
                self.covered = 1
        self.covered -= 1
        self.remaining -= 1


def slowest_rank_ms(torch, dist, ms, world, device):
    """Per-step time of the slowest rank (the ranks are independent replicas; the job is as slow as
    its slowest one).  `dist` is an initialised torch.distributed or None when world == 1."""
    if world <= 1:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbps(step_bytes, world, ms):
    """Bytes moved by all replicas in one step over the slowest rank's step time."""
    return world * step_bytes / (ms * 1e-3) / 1e9


def time_steps(torch, dist, run_step, steps, warmup, device_index, world, min_repeats=1, min_seconds=0.0):
    """W warm-up steps, then R repetitions of exactly K steps, each repetition between its own pair of CUDA
    events on the current stream, the whole timed region bracketed by a barrier and a device synchronise on
    both sides.  R is at least `min_repeats` and large enough for the region to last `min_seconds`.
    Returns (median ms per step: max over ranks, clocks, statistics of the repetitions)."""
    begin = getattr(run_step, "begin", lambda n: None)
    begin(warmup)
    for i in range(warmup):
        run_step(i)
    torch.cuda.synchronize()
    repeats = max(1, min_repeats)
    if min_seconds > 0:
        # one untimed repetition to size the region
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        begin(steps)
        a.record()
        for i in range(steps):
            run_step(warmup + i)
        b.record()
        torch.cuda.synchronize()
        repeats = max(repeats, int(np.ceil(min_seconds * 1e3 / max(1e-3, a.elapsed_time(b)))))
        repeats = min(repeats, 2000)
    if world > 1:
        r = torch.tensor([repeats], device="cuda", dtype=torch.int64)
        dist.all_reduce(r, op=dist.ReduceOp.MAX)
        repeats = int(r.item())
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    sampler.start()
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(repeats)]
    for start, stop in events:
        begin(steps)
        start.record()
        for i in range(steps):
            run_step(warmup + i)
        stop.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    per_step = np.array([start.elapsed_time(stop) / steps for start, stop in events])
    ms = float(np.median(per_step))
    stats = {"repeats": repeats, "steps_per_repeat": steps, "median_ms": round(ms, 5), "min_ms": round(float(per_step.min()), 5),
             "max_ms": round(float(per_step.max()), 5), "timed_region_ms": round(float(per_step.sum() * steps), 2)}
    if world > 1:
        ms = slowest_rank_ms(torch, dist, ms, world, "cuda")
        dist.barrier()
    torch.cuda.synchronize()
    return ms, clocks, stats


def full_bn_bytes(layers):
    """Full BN: 3 passes forward + 5 backward; with the fused residual + ReLU 4 + 9 (residual read three times,
    dresidual written, the second backward pass re-reads x, residual and dy)."""
    return sum(l.count * ((13 if l.rule == "relu" else 8) * l.elems * l.ebytes + 32 * l.C) for l in layers)


def buffer_sets(layers):
    """Rotating buffer sets, so that no tensor is reused before more than 2x L2 (126 MB) of other data went by."""
    bytes_per_tensor_set = sum(4 * l.elems * l.ebytes for l in layers)
    return 2 if bytes_per_tensor_set >= 512e6 else min(8, max(2, int(np.ceil(512e6 / bytes_per_tensor_set))))


def measure_workload(torch, dist, bns, args, layers, inputs, local, world, seconds, layer_seconds, per_layer=True,
                     warm=True, dev=None):
    """Times one workload: the whole step (sampled), the same layers through full BN, and each layer alone;
    every number is the median over at least 30 repetitions of `--steps` steps.  Returns (dict, device layers)."""
    nhwc = args.layout == "nhwc"
    sets = buffer_sets(layers)
    if dev is None:
        dev = [DeviceLayer(l, h, sets, torch, bns, nhwc=nhwc) for l, h in zip(layers, inputs)]
    full = ([DeviceLayer(l, h, sets, torch, bns, full_bn=True, nhwc=nhwc) for l, h in zip(layers, inputs)]
            if args.full_bn else [])

    def step(i):
        for d in dev:
            for _ in range(d.layer.count):
                d.step(i)

    def full_step(i):
        for d in full:
            for _ in range(d.layer.count):
                d.step(i)

    def runner(fn, nsets=sets):
        g = capture_steps(torch, fn, nsets) if args.graph else None
        return (GraphedSteps(g, fn, nsets) if g else fn), g is not None

    step_bytes = sum(l.count * l.algorithmic_bytes() for l in layers)
    run, graphed = runner(step)
    for attempt in range(2):
        ms, clocks, stats = time_steps(torch, dist, run, args.steps, args.warmup, local, world, 30, seconds)
        if not clocks_rejected(clocks):
            break
    res = {"ms_per_step": round(ms, 5), "value": round(whole_job_gbps(step_bytes, world, ms), 1), "timing": stats,
           "clocks": clocks, "algorithmic_bytes_per_step": step_bytes, "graphed": graphed, "sets": sets}
    if warm:
        # the same step on ONE buffer set, back to back: whatever fits in L2 (126 MB) is found there
        wrun, _ = runner(lambda i: step(0), 1)
        wms, _, wstats = time_steps(torch, dist, wrun, args.steps, args.warmup, local, world, 30, seconds / 2)
        res["warm_l2"] = {"ms_per_step": round(wms, 5), "value": round(whole_job_gbps(step_bytes, world, wms), 1),
                          "min_ms": wstats["min_ms"], "note": "one buffer set reused every step (no rotation)"}
    layer_info = {}
    if per_layer:
        for d in dev:
            lms, _, lst = time_steps(torch, dist, runner(d.step)[0], args.steps, args.warmup, local, world, 30, layer_seconds)
            layer_info[d.layer.name] = {"ms": round(lms, 5), "min_ms": lst["min_ms"],
                                        "gbps": round(d.layer.algorithmic_bytes() / lms / 1e6, 1),
                                        "algorithmic_bytes": d.layer.algorithmic_bytes(), "count": d.layer.count}
    if full:
        fms, _, fst = time_steps(torch, dist, runner(full_step)[0], args.steps, args.warmup, local, world, 30, seconds / 2)
        fbytes = full_bn_bytes(layers)
        res["full_bn"] = {"ms_per_step": round(fms, 5), "min_ms": fst["min_ms"], "gbps": round(fbytes / fms / 1e6, 1),
                          "algorithmic_bytes": fbytes, "speedup_sampled_vs_full": round(fms / ms, 4)}
        if per_layer:
            for d in full:
                lms, _, _ = time_steps(torch, dist, runner(d.step)[0], args.steps, args.warmup, local, world, 30, layer_seconds)
                layer_info[d.layer.name]["full_bn_ms"] = round(lms, 5)
                layer_info[d.layer.name]["speedup_vs_full_bn"] = round(lms / layer_info[d.layer.name]["ms"], 4)
            # the paper's estimation errors (Sec. 5.1, "Correlation Analysis"): E_mu = ||mu_s - mu||_2 and
            # E_sigma = ||sigma_s - sigma||_2 between the sampled statistics and those of the whole batch,
            # from the vectors the two forward calls above left behind (diagnostic; synthetic activations)
            torch.cuda.synchronize()
            for d, f in zip(dev, full):
                if d.relu or d.nhwc:
                    continue                      # that path keeps its statistics in tensors of its own
                sigma_s, sigma = 1.0 / d.invstd.double(), 1.0 / f.invstd.double()     # sqrt(var + eps) each
                layer_info[d.layer.name]["estimation_error"] = {
                    "E_mu": round(float((d.mean.double() - f.mean.double()).norm()), 6),
                    "E_sigma": round(float((sigma_s - sigma).norm()), 6), "channels": d.layer.C}
    res["per_layer"] = layer_info
    return res, dev


OTHER_CONFIGS = ["tiny", "cifar", "vdn", "resnet50", "fs_vdn", "fs_relu"]


def run_ours(args):
    import torch
    from paper_1810_10962_b200 import bns
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run --nproc-per-node N")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    bns.load()
    for item in args.tune:
        name, value = item.split("=")
        bns.set_tuning(name, int(value))
    layers, seeds = selected_layers(args)
    hosts = [host_inputs(l, s) for l, s in zip(layers, seeds)]
    nhwc = args.layout == "nhwc"
    peak, peak_source = measured_hbm_peak()
    sets = buffer_sets(layers)

    # ---- kernel-level events of the library on (K eager steps): the roofline of the dominant kernel
    dev = [DeviceLayer(l, h, sets, torch, bns, nhwc=nhwc) for l, h in zip(layers, hosts)]

    def step(i):
        for d in dev:
            for _ in range(d.layer.count):
                d.step(i)

    bns.profile_enable(False)
    for i in range(args.warmup):     # warm-up outside the profiled window
        step(i)
    bns.profile_enable(True)
    bns.launch_count_reset()
    ms_events, _, _ = time_steps(torch, dist, step, args.steps, 0, local, world)
    launches = bns.launch_count()
    kernel_times = {}
    for kind in range(bns.KERNEL_KINDS):
        n, tot = bns.profile_read(kind)
        if n:
            kernel_times[bns.kernel_name(kind)] = {"launches": n, "total_ms": round(tot, 4), "avg_us": round(1e3 * tot / n, 3)}
    bns.profile_enable(False)

    # ---- the reported value: median over >= 30 repetitions of the K steps, per-kernel events off
    main, dev = measure_workload(torch, dist, bns, args, layers, hosts, local, world, args.seconds, args.seconds / 4,
                                 dev=dev)
    ms_plain, value = main["ms_per_step"], main["value"]
    step_bytes = main["algorithmic_bytes_per_step"]

    # ---- roofline of the dominant kernel: backward pass 1 reads dy and x and writes dx (3 E b per launch)
    roofline = None
    kt = kernel_times.get("col_bwd_reduce_kernel")
    if kt:
        launches_per_step = sum(l.count for l in layers)
        algo = sum(l.count * 3 * l.elems * l.ebytes for l in layers) / launches_per_step
        achieved = algo / (kt["avg_us"] * 1e-6) / 1e9
        roofline = {"kernel": "col_bwd_reduce_kernel", "bound": "hbm", "achieved": round(achieved, 1), "peak": peak,
                    "unit": "GB/s", "frac": round(achieved / peak, 4),
                    "traffic": BWD_REDUCE_DRAM_TRAFFIC_BYTES if args.workload == "resnet18_stage1" and not args.only else None,
                    "algorithmic_bytes_per_launch": int(algo), "avg_launch_us": kt["avg_us"], "peak_source": peak_source,
                    "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4)}

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if args.e2e and rank == 0 and not nhwc:
        e2e = run_e2e(torch, bns, layers, hosts, max(2, min(args.steps, args.e2e_steps)))
    if world > 1:
        dist.barrier()

    # ---- the other configurations of the benchmark spec, each a bounded measurement with its own clock record
    others = None
    if args.other_configs and world == 1 and args.workload == "resnet18_stage1" and not args.only and not nhwc:
        del dev
        torch.cuda.empty_cache()
        others = {}
        oargs = argparse.Namespace(**vars(args))
        oargs.steps = min(args.steps, 20)          # bounded: these are side measurements of the same run
        for name in OTHER_CONFIGS:
            olayers = workload_layers(name)
            oin = [device_inputs(l, layer_seed(name, i), torch) for i, l in enumerate(olayers)]
            res, odev = measure_workload(torch, dist, bns, oargs, olayers, oin, local, world, args.seconds / 2,
                                         args.seconds / 8, warm=name in ("tiny", "cifar", "vdn"))
            res["steps_per_repeat"] = oargs.steps
            res["frac_of_hbm_peak"] = round(res["value"] / peak, 4)
            res["frac_of_nominal_8TBps"] = round(res["value"] / NOMINAL_HBM_GBS, 4)
            res["layers"] = [f"{l.name}:{l.N}x{l.C}x{l.H}x{l.W}:{l.dtype}:x{l.count}" for l in olayers]
            res["data"] = "synthetic, drawn on the device with the recipe of the main workload"
            others[name] = res
            del odev, oin
            torch.cuda.empty_cache()

    # ---- the oracle on the host cores, bounded sample
    cpu = run_cpu_baseline(layers, hosts, args.cpu_seconds) if (rank == 0 and world == 1 and args.cpu_seconds > 0) else None

    if rank == 0:
        first = layers[0]
        line = {
            "metric": "sampled_bn_fwd_bwd_algorithmic_gbps", "value": round(value, 1), "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_plain, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": first.dtype, "data": "synthetic",
            "config": {"workload": args.workload + (f" (only {args.only})" if args.only else ""),
                       "layers": [f"{l.name}:{l.N}x{l.C}x{l.H}x{l.W}:{l.dtype}:x{l.count}" for l in layers],
                       "step": "forward+backward of every layer", "algorithmic_bytes_per_step": step_bytes,
                       "cache": f"inputs larger than L2; {sets} buffer sets rotated", "replicas": world, "layout": args.layout,
                       "launch": f"CUDA graph replay, {sets} steps per graph" if main["graphed"] else "eager launches",
                       "value_is": "median over the repetitions of the K-step loop", "tuning": args.tune},
            "timing": main["timing"], "min_ms_per_step": main["timing"]["min_ms"], "repeats": main["timing"]["repeats"],
            "warm_l2": main.get("warm_l2"),
            "frac_of_hbm_peak": round(value / world / peak, 4), "hbm_peak_gbs": peak, "hbm_peak_source": peak_source,
            "frac_of_nominal_8TBps": round(value / world / NOMINAL_HBM_GBS, 4),
            "clocks": main["clocks"], "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu,
            "kernels": kernel_times, "ms_per_step_with_kernel_events": round(ms_events, 5),
            "per_layer": main["per_layer"], "full_bn": main.get("full_bn"),
            "other_configs": others,
            "paper_context": "overall training speed-up up to 20% (ResNet-18: BS +16.5%, VDN +13.8%, FS +10.7% on 2x V100, "
                             "TensorFlow); not comparable to a kernel GB/s",
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(torch, bns, layers, hosts, steps):
    """Same metric through bns_forward_backward_host: pinned host tensors in, pinned host tensors out."""
    items, h2d, d2h = [], 0, 0
    for l, h in zip(layers, hosts):
        if l.rule in ("virtual", "mixed", "relu"):
            return None      # the host entry point keeps xv on the device; not measured end to end
        dt = torch.float32 if l.dtype == "f32" else torch.bfloat16
        pin = lambda a: torch.from_numpy(a).to(dt).pin_memory()
        x, dy = pin(h["x"]), pin(h["dy"])
        y, dx = torch.empty_like(x).pin_memory(), torch.empty_like(x).pin_memory()
        vec = [torch.empty(l.C, dtype=torch.float32).pin_memory() for _ in range(4)]
        gamma, beta = torch.from_numpy(h["gamma"]).pin_memory(), torch.from_numpy(h["beta"]).pin_memory()
        if l.rule == "batch":
            sp = bns.Sampling.batch(h["sample_idx"])
        elif l.rule == "feature":
            sp = bns.Sampling.feature(l.kw["ph"], l.kw["pw"], h["offsets"])
        else:
            sp = bns.Sampling.full()
        arena = torch.empty(bns.host_arena_bytes(x.shape, dt, sp), dtype=torch.uint8, device="cuda")
        items.append((l, x, dy, gamma, beta, sp, y, dx, vec, arena))
        h2d += l.count * (2 * l.elems * l.ebytes + 8 * l.C)
        d2h += l.count * (2 * l.elems * l.ebytes + 16 * l.C)

    def step():
        for l, x, dy, gamma, beta, sp, y, dx, vec, arena in items:
            for _ in range(l.count):
                bns.forward_backward_host(x, dy, gamma, beta, EPS, sp, y, dx, vec[0], vec[1], vec[2], vec[3], arena)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        step()
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps
    step_bytes = sum(l.count * l.algorithmic_bytes() for l in layers)
    return {"value": round(step_bytes / ms / 1e6, 2), "unit": "GB/s", "ms_per_step": round(ms, 4), "steps": steps,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "entry": "bns_forward_backward_host (pinned host buffers, copies inside the timed region)"}


# ----------------------------------------------------------------------------- the oracle arm
def oracle_sample(layers, hosts, seconds):
    """Runs the oracle (forward+backward) on a subset of channels of every layer, sized to take roughly
    `seconds` in total.  Returns (algorithmic bytes of the sample, elapsed seconds, description)."""
    import oracle as O
    threads = O.threads()

    def run(l, h, channels):
        if l.rule == "batch":
            sp = O.Sampling.batch(h["sample_idx"])
        elif l.rule == "feature":
            sp = O.Sampling.feature(l.kw["ph"], l.kw["pw"], h["offsets"])
        elif l.rule == "virtual":
            sp = O.Sampling.virtual(l.kw["nv"])
        else:
            sp = O.Sampling.full()
        ch = np.asarray(channels, dtype=np.int32)
        if l.rule == "relu":
            sp = O.Sampling.feature(l.kw["ph"], l.kw["pw"], h["offsets"])
            t0 = time.perf_counter()
            f = O.forward_relu(h["x"], h["residual"], h["gamma"], h["beta"], EPS, sp, channels=ch)
            O.backward_relu(h["x"], h["dy"], h["gamma"], f, EPS, sp, channels=ch)
            return time.perf_counter() - t0
        if l.rule == "mixed":
            sp = O.Sampling.feature(l.kw["ph"], l.kw["pw"], h["offsets"])
            t0 = time.perf_counter()
            f = O.forward_mixed(h["x"], h["xv"], h["gamma"], h["beta"], EPS, l.kw["mix"], sp, channels=ch)
            O.backward_mixed(h["x"], h["xv"], h["dy"], None, h["gamma"], f, EPS, l.kw["mix"], sp, channels=ch)
            return time.perf_counter() - t0
        t0 = time.perf_counter()
        f = O.forward(h["x"], h["gamma"], h["beta"], EPS, sp, xv=h.get("xv"), channels=ch)
        O.backward(h["x"], h["dy"], h["gamma"], f.mean, f.var, EPS, sp, xv=h.get("xv"), channels=ch)
        return time.perf_counter() - t0

    # calibrate on one channel per thread of the first layer, then share the budget by layer size
    l0, h0 = layers[0], hosts[0]
    probe = list(range(min(l0.C, threads)))
    t_probe = run(l0, h0, probe)
    per_channel_elem = t_probe / (len(probe) * l0.N * l0.H * l0.W)          # seconds per element of a channel
    total_elem_channels = sum(l.count * l.N * l.H * l.W * l.C for l in layers)
    frac = min(1.0, seconds / max(1e-9, per_channel_elem * total_elem_channels))
    elapsed, sample_bytes, parts = 0.0, 0.0, []
    for l, h in zip(layers, hosts):
        nch = int(min(l.C, max(min(l.C, threads), round(frac * l.C))))
        ch = np.linspace(0, l.C - 1, nch).round().astype(np.int32)
        ch = np.unique(ch)
        elapsed += l.count * run(l, h, ch)
        sample_bytes += l.count * l.algorithmic_bytes() * (len(ch) / l.C)
        parts.append(f"{l.name}: {len(ch)} of {l.C} channels" + (f" x{l.count} (timed once)" if l.count > 1 else ""))
    return sample_bytes, elapsed, "; ".join(parts), threads


def run_cpu_baseline(layers, hosts, seconds):
    sample_bytes, elapsed, what, threads = oracle_sample(layers, hosts, seconds)
    return {"value": round(sample_bytes / elapsed / 1e9, 4), "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"forward+backward of {what}; {elapsed:.1f} s of wall time; channels are independent, so the "
                      f"rate extrapolates to the whole layer", "host_cpus": os.cpu_count()}


def run_reference(args):
    """The oracle as it stands on the host cores: each step is a bounded channel sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers, seeds = selected_layers(args)
    hosts = [host_inputs(l, s) for l, s in zip(layers, seeds)]
    # exactly the requested steps; the channel sample of a step is sized so that the whole run takes about 90 s at
    # most (never less than one channel per thread and layer)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_step = min(20.0, 90.0 / (steps + warmup))
    for _ in range(warmup):
        oracle_sample(layers, hosts, per_step)
    tot_bytes, tot_s, what, threads = 0.0, 0.0, "", 1
    for _ in range(steps):
        b, s, what, threads = oracle_sample(layers, hosts, per_step)
        tot_bytes += b
        tot_s += s
    value = round(tot_bytes / tot_s / 1e9, 4)
    first = layers[0]
    line = {
        "impl": "reference", "metric": "sampled_bn_fwd_bwd_algorithmic_gbps", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": round(1e3 * tot_s / steps, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload,
                   "layers": [f"{l.name}:{l.N}x{l.C}x{l.H}x{l.W}:{l.dtype}:x{l.count}" for l in layers],
                   "step": "forward+backward of a channel sample of every layer (CPU oracle, double precision)"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="resnet18_stage1",
                    choices=["resnet18_stage1", "cifar", "vdn", "resnet50", "fs_vdn", "fs_relu", "tiny"])
    ap.add_argument("--only", default=None, help="comma-separated layer names: run just these layers of the workload")
    ap.add_argument("--tune", action="append", default=[], metavar="NAME=VALUE",
                    help="launch-shape knob of the library (bns_set_tuning), e.g. --tune pdl=0")
    ap.add_argument("--no-full-bn", dest="full_bn", action="store_false", help="skip the full-BN comparison")
    ap.add_argument("--layout", choices=["nchw", "nhwc"], default="nchw",
                    help="tensor layout of the timed calls (nhwc: the channels-last entry points)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="time eager launches instead of replaying a CUDA graph of the step")
    ap.add_argument("--no-e2e", dest="e2e", action="store_false", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--seconds", type=float, default=0.6,
                    help="least duration of the main timed region (the K-step loop is repeated, 30 times at least)")
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="skip the bounded measurements of the other configurations (CIFAR sweep, VDN, ResNet-50 sweep, ...)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the oracle baseline (0 = skip)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
