"""GPU parity: the C ABI against the CPU oracle, element by element, on the five benchmark
configurations and on the edge cases."""
import numpy as np
import pytest

import bns_inputs as I
import oracle as O
from helpers import Case, compare, gpu_sampling, make_case, run_gpu, _to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["onchip", "streaming"])
def execution_path(request):
    """Every case runs twice: with the one-launch on-chip path taken by every layer that fits it (the limits
    that the library applies by default - small tensors only, not for small sampled sets - are lifted, so
    the mid-sized layers and every rule exercise it too; the rest streams anyway), and with that path
    switched off (everything goes through the streaming kernels and their partial sums)."""
    from paper_1810_10962_b200 import bns
    bns.set_tuning("slab", 1 if request.param == "onchip" else 0)
    bns.set_tuning("slab_max_mb", 1 << 20)
    bns.set_tuning("slab_small_sets", 1)
    yield request.param
    bns.set_tuning("slab", 1)
    bns.set_tuning("slab_max_mb", DEFAULT_SLAB_MAX_MB)
    bns.set_tuning("slab_small_sets", 0)


DEFAULT_SLAB_MAX_MB = 6


# ----------------------------------------------------------------------------- config 1: tiny
@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=2, contiguous=False)),
    ("batch", dict(k=2, contiguous=True)),
    ("feature", dict(ph=3, pw=3, offset_mode=0)),
    ("feature", dict(ph=2, pw=5, offset_mode=1)),
    ("feature", dict(ph=4, pw=1, offset_mode=2)),
    ("virtual", dict(nv=2)),
    ("virtual", dict(nv=1, with_dyv=False)),
    ("full", dict()),
])
def test_config1_tiny(rule, kw):
    case = make_case(8, 16, 8, 8, rule, seed=1811, generator="tiny", **kw)
    compare(case, run_gpu(case))


# ----------------------------------------------------------------------------- config 2: CIFAR sweep
@pytest.mark.parametrize("C,H", I.cifar_resnet_layers())
@pytest.mark.parametrize("mode", [0, 2])
def test_config2_cifar_feature_sampling(C, H, mode):
    case = make_case(128, C, H, H, "feature", seed=1812, ph=4, pw=4, offset_mode=mode)
    compare(case, run_gpu(case))


# ----------------------------------------------------------------------------- config 3: ResNet-18 stage 1, full size
@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=32, contiguous=True)),
    ("feature", dict(ph=8, pw=8, offset_mode=0)),
    ("full", dict()),
])
def test_config3_resnet18_stage1_full_size(rule, kw):
    case = make_case(256, 64, 56, 56, rule, seed=1813, **kw)
    compare(case, run_gpu(case))                         # every channel, every element


# ----------------------------------------------------------------------------- config 4: VDN, bf16 activations
def test_config4_vdn_bf16():
    case = make_case(256, 128, 28, 28, "virtual", seed=1814, dtype="bf16", nv=2, xv_dtype="f32", with_dyv=False)
    compare(case, run_gpu(case))                         # every channel, every element


# ----------------------------------------------------------------------------- config 5: ResNet-50 sweep, bf16
def _distinct_resnet50():
    return sorted(set(I.resnet50_bn_layers()), key=lambda t: (-t[1], t[0]))


def _channels_to_check(C, HW, positions_per_tile, spread=24, straddlers=24):
    """Channels spread over the layer plus channels whose map straddles two tiles of the streaming kernels
    (a tile is `positions_per_tile` consecutive positions of a sample row): those receive partial sums
    from two blocks per row chunk."""
    straddling = [c for c in range(C) if (c * HW) // positions_per_tile != ((c + 1) * HW - 1) // positions_per_tile]
    if len(straddling) > straddlers:
        straddling = [straddling[i] for i in np.linspace(0, len(straddling) - 1, straddlers).round().astype(int)]
    picked = set(straddling) | set(np.linspace(0, C - 1, min(C, spread)).round().astype(int).tolist())
    return sorted(int(c) for c in picked)


@pytest.mark.parametrize("C,H", _distinct_resnet50())
def test_config5_resnet50_layers_full_size(C, H):
    p = max(1, H // 8)
    case = make_case(256, C, H, H, "feature", seed=1815, dtype="bf16", ph=p, pw=p, offset_mode=0)
    channels = _channels_to_check(C, H * H, positions_per_tile=256 * 8)      # 256 threads x 8 bf16 per thread
    assert len(channels) >= min(C, 24)
    compare(case, run_gpu(case), channels=channels)


# ----------------------------------------------------------------------------- edge cases
EDGE = [
    # odd everything: one element per vector
    dict(N=3, C=3, H=5, W=7, rule="feature", ph=5, pw=7),                  # patch = whole map
    dict(N=3, C=3, H=5, W=7, rule="feature", ph=1, pw=1, offset_mode=2),   # one point per map
    dict(N=5, C=7, H=3, W=3, rule="batch", k=1),
    dict(N=5, C=7, H=3, W=3, rule="batch", k=5, contiguous=False),         # ratio 1
    dict(N=1, C=4, H=6, W=6, rule="full"),
    dict(N=2, C=130, H=1, W=1, rule="batch", k=1),                         # fully connected layer: HW = 1
    dict(N=64, C=40, H=1, W=1, rule="full"),
    dict(N=9, C=12, H=2, W=2, rule="virtual", nv=3),                       # HW smaller than a vector
    dict(N=4, C=6, H=7, W=7, rule="feature", ph=3, pw=2, offset_mode=1, dtype="bf16"),   # P*2 % 16 != 0
    dict(N=4, C=8, H=7, W=7, rule="batch", k=3, contiguous=False, dtype="bf16"),         # 98-byte maps
    dict(N=6, C=16, H=14, W=14, rule="full", dtype="bf16"),
    dict(N=6, C=16, H=14, W=14, rule="virtual", nv=2, dtype="bf16", xv_dtype="bf16"),
    dict(N=70, C=5, H=33, W=31, rule="batch", k=9),                        # several row chunks, ragged tile tail
    dict(N=37, C=300, H=4, W=4, rule="feature", ph=2, pw=3, offset_mode=2),
]


@pytest.mark.parametrize("spec", EDGE, ids=lambda s: "-".join(f"{k}{v}" for k, v in s.items()))
def test_edge_cases(spec):
    spec = dict(spec)
    dims = [spec.pop(k) for k in ("N", "C", "H", "W")]
    rule = spec.pop("rule")
    case = make_case(*dims, rule, seed=77, generator="tiny", **spec)
    compare(case, run_gpu(case))


def test_patch_at_every_border():
    N, C, H, W = 4, 5, 9, 11
    for oh, ow in [(0, 0), (0, W - 4), (H - 3, 0), (H - 3, W - 4)]:
        case = make_case(N, C, H, W, "feature", seed=78, generator="tiny", ph=3, pw=4)
        case.offsets = np.array([[oh, ow]], np.int32)
        compare(case, run_gpu(case))


def test_full_bn_entry_point_equals_full_rule():
    case = make_case(16, 24, 10, 10, "full", seed=79)
    a, b = run_gpu(case, use_full_bn_entry=True), run_gpu(case)
    for key in ("y", "mean", "invstd", "dx", "dgamma", "dbeta"):
        assert np.array_equal(getattr(a, key), getattr(b, key)), key
    compare(case, a)


def test_ratio_one_matches_full_bn_on_gpu():
    """Batch Sampling with every sample and Feature Sampling with the whole map are ordinary BN."""
    full = make_case(12, 10, 6, 6, "full", seed=80)
    gf = run_gpu(full)
    bs = make_case(12, 10, 6, 6, "batch", seed=80, k=12)
    fs = make_case(12, 10, 6, 6, "feature", seed=80, ph=6, pw=6)
    for case in (bs, fs):
        g = run_gpu(case)
        compare(case, g)
        np.testing.assert_allclose(g.y, gf.y, rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(g.dx, gf.dx, rtol=1e-4, atol=1e-5)


# ----------------------------------------------------------------------------- selection is bit-exact
@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=5, contiguous=False)), ("batch", dict(k=4, contiguous=True)),
    ("feature", dict(ph=3, pw=2, offset_mode=0)), ("feature", dict(ph=3, pw=2, offset_mode=1)),
    ("feature", dict(ph=1, pw=4, offset_mode=2)), ("virtual", dict()), ("full", dict()),
])
def test_selection_mask_bit_exact(rule, kw):
    from paper_1810_10962_b200 import bns
    case = make_case(11, 6, 7, 9, rule, seed=81, generator="tiny", **kw)
    x = _to_device(case.x, "f32")
    mask = bns.selection_mask(x, gpu_sampling(case)).cpu().numpy()
    assert np.array_equal(mask, O.selection_mask(11, 6, 7, 9, case.oracle_sampling()))


def test_selection_sentinel_through_the_statistics():
    """x = 1 exactly on S, 0 elsewhere -> the GPU statistics must be mean 1, var 0 (invstd eps^-1/2)."""
    for rule, kw in [("batch", dict(k=3, contiguous=False)), ("feature", dict(ph=2, pw=3, offset_mode=2))]:
        case = make_case(10, 6, 8, 8, rule, seed=82, generator="tiny", **kw)
        case.x = O.selection_mask(10, 6, 8, 8, case.oracle_sampling()).astype(np.float32)
        g = run_gpu(case)
        assert np.array_equal(g.mean, np.ones(6, np.float32))
        np.testing.assert_allclose(g.invstd, np.float32(1e-5) ** -0.5, rtol=1e-6)


# ----------------------------------------------------------------------------- determinism
@pytest.mark.parametrize("rule,kw", [("batch", dict(k=8)), ("feature", dict(ph=4, pw=4)), ("full", dict())])
def test_runs_are_bit_identical(rule, kw):
    import torch
    case = make_case(64, 32, 28, 28, rule, seed=83, **kw)
    a, b = run_gpu(case), run_gpu(case)
    for key in a.raw:
        assert torch.equal(a.raw[key], b.raw[key]), key


# ----------------------------------------------------------------------------- device-resident offsets are checked
def test_bad_device_offsets_raise_flag_and_stay_in_bounds():
    import torch
    from paper_1810_10962_b200 import bns
    case = make_case(4, 3, 6, 6, "feature", seed=84, generator="tiny", ph=2, pw=2, offset_mode=1)
    x = _to_device(case.x, "f32")
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    good = torch.from_numpy(case.offsets).cuda()
    sp = bns.Sampling.feature(2, 2, good, bns.OFF_PER_SAMPLE)
    ws = bns.new_workspace(x, sp)
    bns.forward(x, gamma, beta, 1e-5, sp, workspace=ws)
    assert bns.workspace_status(ws) == 0
    bad = good.clone()
    bad[1, 0] = 99
    bad[2, 1] = -3
    sp_bad = bns.Sampling.feature(2, 2, bad, bns.OFF_PER_SAMPLE)
    y, mean, invstd = bns.forward(x, gamma, beta, 1e-5, sp_bad, workspace=ws)
    assert bns.workspace_status(ws) & bns.FLAG_BAD_OFFSET
    # clamped into range: same as the nearest valid offsets
    clamped = case.offsets.copy()
    clamped[1, 0], clamped[2, 1] = 4, 0
    case.offsets = clamped
    f = O.forward(case.x, case.gamma, case.beta, 1e-5, case.oracle_sampling())
    np.testing.assert_allclose(mean.cpu().numpy(), f.mean, atol=1e-5)


# ----------------------------------------------------------------------------- launch-shape knobs change no bits they should not
@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=6)), ("feature", dict(ph=3, pw=3, offset_mode=2)), ("virtual", dict(nv=2)), ("full", dict()),
])
def test_programmatic_dependent_launch_changes_nothing(rule, kw):
    """With and without programmatic dependent launch the kernels run the same arithmetic in the same
    order, so the results must be identical bit for bit."""
    import torch
    from paper_1810_10962_b200 import bns
    case = make_case(40, 24, 20, 20, rule, seed=85, **kw)
    try:
        bns.set_tuning("pdl", 0)
        a = run_gpu(case)
    finally:
        bns.set_tuning("pdl", 1)
    b = run_gpu(case)
    compare(case, b)
    for key in a.raw:
        assert torch.equal(a.raw[key], b.raw[key]), key


@pytest.mark.parametrize("target", [37, 148, 4736])
def test_other_grid_shapes_still_match_the_oracle(target):
    """Splitting the rows into more or fewer chunks reorders sums but must stay within tolerance."""
    from paper_1810_10962_b200 import bns
    try:
        bns.set_tuning("target_blocks", target)
        bns.set_tuning("stat_target_blocks", target)
        for rule, kw in [("batch", dict(k=9)), ("feature", dict(ph=5, pw=3)), ("full", dict())]:
            case = make_case(70, 12, 33, 31, rule, seed=86, **kw)
            compare(case, run_gpu(case))
    finally:
        bns.set_tuning("target_blocks", 0)
        bns.set_tuning("stat_target_blocks", 0)


@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=3, contiguous=False)), ("batch", dict(k=2)), ("feature", dict(ph=3, pw=3, offset_mode=0)),
    ("feature", dict(ph=2, pw=4, offset_mode=2)), ("virtual", dict(nv=2)), ("virtual", dict(nv=1, with_dyv=False)),
])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_sampled_sets_both_paths(rule, kw, dtype):
    """A small sampled set is handled by one block per channel, a large one through partial sums and a
    finalize launch; forcing either path on the same case must match the oracle."""
    from paper_1810_10962_b200 import bns
    kw = dict(kw)
    if rule == "virtual":
        kw["xv_dtype"] = dtype
    case = make_case(24, 20, 14, 14, rule, seed=87, dtype=dtype, **kw)
    try:
        for direct_max in (0, 1 << 20):
            bns.set_tuning("direct_max", direct_max)
            compare(case, run_gpu(case))
    finally:
        bns.set_tuning("direct_max", 8192)


# ----------------------------------------------------------------------------- seeded random sweep
def _random_specs(count, seed):
    rng = np.random.default_rng(seed)
    specs = []
    for i in range(count):
        N = int(rng.integers(1, 40))
        C = int(rng.integers(1, 70))
        H = int(rng.integers(1, 20))
        W = int(rng.integers(1, 20))
        rule = ["batch", "feature", "virtual", "full"][i % 4]
        dtype = "bf16" if rng.random() < 0.4 else "f32"
        kw = {}
        if rule == "batch":
            kw = dict(k=int(rng.integers(1, N + 1)), contiguous=bool(rng.random() < 0.5))
        elif rule == "feature":
            kw = dict(ph=int(rng.integers(1, H + 1)), pw=int(rng.integers(1, W + 1)), offset_mode=int(rng.integers(0, 3)))
        elif rule == "virtual":
            kw = dict(nv=int(rng.integers(1, 4)), xv_dtype=dtype if rng.random() < 0.5 else "f32",
                      with_dyv=bool(rng.random() < 0.5))
        specs.append((N, C, H, W, rule, dtype, kw, 1000 + i))
    return specs


@pytest.mark.parametrize("spec", _random_specs(48, 2024), ids=lambda s: f"{s[4]}-{s[5]}-{s[0]}x{s[1]}x{s[2]}x{s[3]}")
def test_random_shapes_and_rules(spec):
    """Shapes nobody tuned for: odd sizes, one sample, one channel, 1x1 maps, patches of any size."""
    N, C, H, W, rule, dtype, kw, seed = spec
    case = make_case(N, C, H, W, rule, seed=seed, dtype=dtype, generator="tiny", **kw)
    compare(case, run_gpu(case))


@pytest.mark.parametrize("ph,pw,mode", [(1, 1, 0), (1, 1, 2), (2, 2, 1), (1, 3, 0), (2, 4, 2), (1, 8, 0)])
@pytest.mark.parametrize("dtype,dims", [("bf16", (70, 37, 7, 9)), ("f32", (33, 130, 14, 14)), ("f32", (5, 3, 4, 8))])
def test_small_patches(ph, pw, mode, dtype, dims):
    """Patches of a few elements: every map contributes one short row segment, channels far apart."""
    case = make_case(*dims, "feature", seed=88, dtype=dtype, generator="tiny", ph=ph, pw=pw, offset_mode=mode)
    compare(case, run_gpu(case))


@pytest.mark.parametrize("rule,kw,N", [("batch", dict(k=4), 20), ("feature", dict(ph=3, pw=3), 20), ("full", dict(), 20),
                                       # 32 samples and more: the two directions of the link overlap by row chunks
                                       ("batch", dict(k=6), 45), ("batch", dict(k=33), 67), ("feature", dict(ph=3, pw=2), 45),
                                       ("feature", dict(ph=10, pw=10), 32), ("batch", dict(k=5, contiguous=False), 40)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_buffer_entry_point(rule, kw, N, dtype):
    """bns_forward_backward_host: pinned host tensors in, pinned host tensors out, copies on the stream."""
    import torch
    from paper_1810_10962_b200 import bns
    from helpers import run_oracle, close_f32, close_bf16, _to_host
    import bns_inputs as I
    case = make_case(N, 12, 10, 10, rule, seed=89, dtype=dtype, **kw)
    dt = torch.float32 if dtype == "f32" else torch.bfloat16

    def pin(a):
        t = torch.from_numpy(a)
        if dtype == "bf16":
            t = torch.from_numpy(I.f32_to_bf16_bits(a).view(np.int16)).view(torch.bfloat16)
        return t.pin_memory()

    x, dy = pin(case.x), pin(case.dy)
    y, dx = torch.empty_like(x).pin_memory(), torch.empty_like(x).pin_memory()
    C = case.x.shape[1]
    mean, invstd, dgamma, dbeta = (torch.empty(C, dtype=torch.float32).pin_memory() for _ in range(4))
    gamma, beta = torch.from_numpy(case.gamma).pin_memory(), torch.from_numpy(case.beta).pin_memory()
    sp = gpu_sampling(case)
    arena = torch.empty(bns.host_arena_bytes(tuple(case.x.shape), dt, sp), dtype=torch.uint8, device="cuda")
    bns.forward_backward_host(x, dy, gamma, beta, case.eps, sp, y, dx, mean, invstd, dgamma, dbeta, arena)
    torch.cuda.synchronize()
    f, b = run_oracle(case)
    tensor_close = close_f32 if dtype == "f32" else close_bf16
    close_f32(mean.numpy(), f.mean, "mean")
    close_f32(invstd.numpy(), f.invstd, "invstd")
    tensor_close(_to_host(y), f.y, "y")
    tensor_close(_to_host(dx), b.dx, "dx")
    close_f32(dgamma.numpy(), b.dgamma, "dgamma")
    close_f32(dbeta.numpy(), b.dbeta, "dbeta")


# ----------------------------------------------------------------------------- the one-launch on-chip path
def _device_case(case):
    import torch
    x, dy = _to_device(case.x, case.dtype), _to_device(case.dy, case.dtype)
    gamma, beta = torch.from_numpy(case.gamma).cuda(), torch.from_numpy(case.beta).cuda()
    return x, dy, gamma, beta


@pytest.mark.parametrize("dims,dtype,rule,kw", [
    ((8, 16, 8, 8), "f32", "batch", dict(k=2)),
    ((128, 16, 32, 32), "f32", "feature", dict(ph=4, pw=4)),
    ((128, 32, 16, 16), "f32", "feature", dict(ph=4, pw=4, offset_mode=2)),
    ((128, 64, 8, 8), "f32", "full", dict()),
    ((256, 128, 28, 28), "bf16", "virtual", dict(nv=2, with_dyv=False)),
    ((256, 256, 14, 14), "bf16", "feature", dict(ph=1, pw=1)),
    ((256, 512, 7, 7), "bf16", "full", dict()),
])
def test_qualifying_layers_take_one_launch_per_direction(dims, dtype, rule, kw, execution_path):
    """Layers whose channel data fits the shared memory of a cluster run forward and backward as one
    kernel each; with the path switched off the same call takes the streaming kernels."""
    from paper_1810_10962_b200 import bns
    case = make_case(*dims, rule, seed=90, dtype=dtype, **kw)
    x, dy, gamma, beta = _device_case(case)
    sp = gpu_sampling(case)
    plans = bns.slab_plan(x, sp, backward=False), bns.slab_plan(x, sp, backward=True)
    ws = bns.new_workspace(x, sp)
    before = bns.launch_count()
    y, mean, invstd = bns.forward(x, gamma, beta, case.eps, sp, workspace=ws)
    bns.backward(x, dy, gamma, mean, invstd, sp, workspace=ws)
    launched = bns.launch_count() - before
    if execution_path == "onchip":
        assert plans[0] is not None and plans[1] is not None
        assert plans[0]["cluster"] <= 8 and plans[1]["smem_bytes"] <= 227 * 1024
        assert launched == 2
    else:
        assert plans == (None, None)
        assert launched >= 4
    assert bns.wait_timeouts() == 0


@pytest.mark.parametrize("cluster_max", [1, 2, 4, 8])
@pytest.mark.parametrize("rule,kw", [
    ("batch", dict(k=5, contiguous=False)), ("feature", dict(ph=3, pw=2, offset_mode=1)), ("virtual", dict(nv=2)),
    ("full", dict()),
])
def test_every_cluster_size_matches_the_oracle(cluster_max, rule, kw, execution_path):
    """The combine across the blocks of a cluster, for 1 to 8 blocks; 37 samples split unevenly."""
    from paper_1810_10962_b200 import bns
    if execution_path != "onchip":
        pytest.skip("this knob belongs to the on-chip path")
    case = make_case(37, 24, 10, 10, rule, seed=91, **kw)
    try:
        bns.set_tuning("slab_cluster_max", cluster_max)
        bns.set_tuning("slab_min_ctas", 1 << 20)        # always grow the cluster to the limit
        compare(case, run_gpu(case))
    finally:
        bns.set_tuning("slab_cluster_max", 8)
        bns.set_tuning("slab_min_ctas", 0)


def test_default_size_limit_of_the_onchip_path():
    """By default only tensors up to a few MiB take the on-chip path (larger ones measured faster through
    the streaming kernels); the limit is a knob."""
    import torch
    from paper_1810_10962_b200 import bns
    bns.set_tuning("slab", 1)
    bns.set_tuning("slab_max_mb", DEFAULT_SLAB_MAX_MB)
    bns.set_tuning("slab_small_sets", 0)
    sp = bns.Sampling.full()
    small = torch.empty(128, 32, 16, 16, device="cuda")                          # 4 MiB
    large = torch.empty(256, 256, 14, 14, device="cuda", dtype=torch.bfloat16)   # 24.5 MiB
    assert bns.slab_plan(small, sp) is not None and bns.slab_plan(small, sp, backward=True) is not None
    assert bns.slab_plan(large, sp) is None
    bns.set_tuning("slab_max_mb", 64)
    assert bns.slab_plan(large, sp) is not None
    # small sampled sets keep their short streaming path unless asked otherwise
    few = bns.Sampling.feature(4, 4, np.array([0, 0]))
    assert bns.slab_plan(small, few) is None
    bns.set_tuning("slab_small_sets", 1)
    assert bns.slab_plan(small, few) is not None
