"""The N > 1 path of bench.py is N independent replicas (BN statistics are local to a GPU in the
paper, so nothing is exchanged): the only cross-rank logic is "time of the slowest rank" and "bytes
of all ranks".  Exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.slowest_rank_ms(torch, dist, 1.0 + rank, world, "cpu")     # rank 1 is the slow one
    dist.barrier()
    out[rank] = (ms, bench.whole_job_gbps(2_000_000_000, world, ms))
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_report_the_slowest_rank_and_the_bytes_of_both():
    world, port = 2, _free_port()
    with mp.Manager() as manager:
        out = manager.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        results = dict(out)
    assert results[0] == results[1]
    ms, gbps = results[0]
    assert ms == 2.0
    assert gbps == pytest.approx(2 * 2.0e9 / 2.0e-3 / 1e9)


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.slowest_rank_ms(torch, None, 3.5, 1, "cpu") == 3.5
    assert bench.whole_job_gbps(1e9, 1, 1.0) == pytest.approx(1000.0)


def test_workloads_match_the_configured_shapes():
    import bench
    import bns_inputs as I
    r50 = bench.workload_layers("resnet50")
    assert sum(l.count for l in r50) == 53 and len(r50) == 12
    assert sum(l.count * l.elems for l in r50) == 2_845_179_904
    assert all(l.kw["ph"] == max(1, l.H // 8) for l in r50)
    r18 = bench.workload_layers("resnet18_stage1")
    assert [(l.N, l.C, l.H, l.W, l.dtype) for l in r18] == [(256, 64, 56, 56, "f32")] * 2
    # (5 + 4r) E b + 32 C
    bs = r18[0]
    assert bs.algorithmic_bytes() == int(round((5 + 4 * 32 / 256) * bs.elems * 4)) + 32 * 64
    assert [(l.C, l.H) for l in bench.workload_layers("cifar")] == I.cifar_resnet_layers()


def _exchange_rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1810_10962_b200 import sync
    rows = torch.full((3, 4), float(rank + 1))
    gathered = sync.all_gather_rows(rows)
    sums = sync.all_reduce_rows(torch.full((2, 4), float(rank + 1)))
    out[rank] = (gathered.tolist(), sums.tolist(), rows.tolist())
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_shared_statistics_exchange_between_two_ranks():
    """The only traffic of the shared-statistics path: an all-gather of the (count, mean, M2) rows in rank
    order and a sum of the backward rows (gloo, CPU tensors; the arithmetic around it runs on the GPU)."""
    world, port = 2, _free_port()
    with mp.Manager() as manager:
        out = manager.dict()
        mp.spawn(_exchange_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        gathered, sums, rows = res[rank]
        assert gathered == [[[1.0] * 4] * 3, [[2.0] * 4] * 3]       # rank-major, same on every rank
        assert sums == [[3.0] * 4] * 2
        assert rows == [[float(rank + 1)] * 4] * 3                  # the input is left alone


def test_reference_arm_prints_one_json_line_with_the_agreed_keys():
    """`bench.py --impl reference` times the CPU oracle; it needs no GPU, so its output format is checked here."""
    import json
    import subprocess
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, cwd=ROOT, timeout=300)
    assert run.returncode == 0, run.stderr
    lines = [l for l in run.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True
    assert d["metric"] == "sampled_bn_fwd_bwd_algorithmic_gbps" and d["value"] > 0 and d["steps"] == 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "tiny" and d["vs_baseline"] is None


def test_other_ranks_of_the_reference_arm_stay_silent():
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2"], capture_output=True, text=True, cwd=ROOT, env=env, timeout=300)
    assert run.returncode == 0 and run.stdout.strip() == ""
