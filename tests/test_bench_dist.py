"""The multi-rank logic of bench.py on CPU (gloo, two ranks): the job's time is the slowest
rank's, the job's throughput the work of all ranks over that time, and the reference arm
runs on rank 0 only."""
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = [40.0, 52.5][rank]                      # rank 1 is the slow one
    ms = bench.reduce_max_ms(local_ms, world, "cpu")
    value = bench.whole_job_tflops(53.45e12, world, ms)
    dist.barrier()
    out[rank] = (ms, value)
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 52.5
    assert abs(value - 2 * 53.45e12 / 52.5e-3 / 1e12) < 1e-9


def _shard_worker(rank, world, port, out):
    """bench.py --shard-heads on CPU: the partition the library gives, every rank's own share of the
    layer's work, a time proportional to that share, the slowest rank's time, the whole layer over it."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2505_18809_b200 import binding as vb, sharding, workloads
    wl = workloads.config("hunyuan-720p")
    host_plan = vb.Plan.from_workload(wl, host_only=True)
    full = host_plan.info.flops_layer
    host_plan.close()
    rank_of_head, rank_flops = sharding.shard_heads(wl, world)
    local = sharding.local_workload(wl, sharding.heads_of_rank(rank_of_head, rank))
    local_plan = vb.Plan.from_workload(local, host_only=True)
    mine = local_plan.info.flops_layer
    local_plan.close()
    local_ms = mine / 1.0e15 * 1e3                       # every rank at 1000 TFLOP/s
    ms = bench.reduce_max_ms(local_ms, world, "cpu")
    value = bench.sharded_job_tflops(full, ms)
    dist.barrier()
    out[rank] = (mine, float(rank_flops[rank]), full, ms, value)
    dist.destroy_process_group()


def test_two_ranks_sharding_one_layer_report_the_whole_layer_over_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    mine = [res[r][0] for r in range(world)]
    full, ms, value = res[0][2], res[0][3], res[0][4]
    for r in range(world):
        assert res[r][0] == pytest.approx(res[r][1], rel=1e-12)     # the rank's plan counts what the partition promised
        assert res[r][2:] == res[0][2:]                             # both ranks report the same job figures
    assert sum(mine) == pytest.approx(full, rel=1e-12)              # the shares add up to the layer
    assert ms == pytest.approx(max(mine) / 1.0e15 * 1e3, rel=1e-12)
    # strong scaling: the whole layer over the slowest rank; below world x the per-rank rate by the imbalance
    assert value == pytest.approx(full / max(mine) * 1000.0, rel=1e-12)
    assert 1000.0 < value <= 1000.0 * world


def test_single_rank_needs_no_process_group():
    assert bench.reduce_max_ms(7.0, 1, "cpu") == 7.0
    assert abs(bench.whole_job_tflops(1e12, 1, 1.0) - 1000.0) < 1e-9


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_window_key_count_matches_the_oracle_mask():
    # the FLOP accounting of sampled sliding rows (bench._window_keys) against the oracle's mask rows
    import oracle
    from paper_2505_18809_b200.workloads import Workload
    wl = Workload("w", (5, 7, 9), 1, 64, (1, 2, 2), (3, 3, 3), 0.5, (1,), 0, False)
    M = oracle.sta_token_mask(wl.grid, wl.tile, wl.window)
    for tok in (0, 17, 100, wl.L - 1):
        assert bench._window_keys(wl, tok) == int(M[tok].sum())


def test_cpu_baseline_flop_accounting_equals_the_plan_accounting_when_every_row_is_sampled():
    """bench.time_oracle counts 4*d*(pairs attended) of the rows it runs; with all rows of a small
    joint workload (text tokens included) that must be the plan's flops_layer."""
    import torch
    from paper_2505_18809_b200 import binding as vb, workloads
    from paper_2505_18809_b200.workloads import Workload
    wl = Workload("acc", (4, 6, 5), 3, 64, (2, 2, 2), (3, 1, 3), 0.5, (0, 1, 2), 3, False, 1, (2, 3, 2), False, 7)
    Q, K, V = workloads.make_qkv(wl, "cpu")
    flops, secs, heads, threads = bench.time_oracle(wl, Q, K, V, wl.L + wl.text, 1e9)
    p = vb.Plan.from_workload(wl, host_only=True)
    want = p.info.flops_layer
    p.close()
    assert heads == wl.heads and threads >= 1 and secs > 0
    assert flops == pytest.approx(want, rel=1e-12)
