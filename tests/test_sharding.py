"""Head-sharded multi-GPU wrapper: the partition (`vorta_shard_heads`, host-only) and the
gather of the ranks' outputs (gloo, world size 2, CPU).  The per-rank compute is stood in
for by the oracle here; the GPU test runs the ranks' shares one after the other on one GPU."""
from __future__ import annotations

import itertools
import os
import socket
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2505_18809_b200 import binding as vb, sharding, workloads  # noqa: E402
from paper_2505_18809_b200.workloads import Workload  # noqa: E402


def head_costs(wl):
    p = vb.Plan.from_workload(wl, host_only=True)
    info = p.info
    p.close()
    per_route = (info.flops_full_head, info.flops_sliding_head, info.flops_coreset_head)
    return np.array([per_route[r] for r in wl.routes])


def best_makespan(cost, n_ranks):
    """Brute force over all assignments (small cases only)."""
    best = float("inf")
    for assign in itertools.product(range(n_ranks), repeat=len(cost)):
        load = np.zeros(n_ranks)
        for h, r in enumerate(assign):
            load[r] += cost[h]
        best = min(best, load.max())
    return best


@pytest.mark.parametrize("routes,n_ranks", [
    ((0, 1, 2, 1, 2, 0, 1), 2), ((0, 0, 0, 1, 1, 2), 3), ((1, 1, 1, 1), 2), ((2, 0), 4), ((0, 1, 2, 2, 1, 0, 1, 1), 3),
])
def test_partition_is_complete_consistent_and_near_optimal(routes, n_ranks):
    wl = Workload("s", (8, 16, 16), len(routes), 128, (4, 8, 8), (3, 3, 3), 0.5, routes, 1, False)
    rank_of_head, rank_flops = sharding.shard_heads(wl, n_ranks)
    cost = head_costs(wl)
    assert rank_of_head.shape == (wl.heads,) and rank_of_head.min() >= 0 and rank_of_head.max() < n_ranks
    load = np.zeros(n_ranks)
    for h, r in enumerate(rank_of_head):
        load[r] += cost[h]
    np.testing.assert_allclose(load, rank_flops, rtol=1e-12)
    # Graham's bound for longest-processing-time-first packing
    opt = best_makespan(cost, n_ranks)
    assert load.max() <= (4.0 / 3.0 - 1.0 / (3.0 * n_ranks)) * opt * (1 + 1e-12)
    # the heaviest head alone is a lower bound nobody can beat
    assert load.max() >= cost.max() * (1 - 1e-12)


def test_partition_rules_on_equal_heads_and_at_the_headline_config():
    wl = Workload("s", (8, 16, 16), 6, 128, (4, 8, 8), (3, 3, 3), 0.5, (0,) * 6, 1, False)
    rank_of_head, _ = sharding.shard_heads(wl, 4)
    # equal costs: heads in ascending order, each to the least loaded rank, lowest rank first
    assert rank_of_head.tolist() == [0, 1, 2, 3, 0, 1]
    wl = workloads.config("hunyuan-720p")
    for n in (1, 2, 4, 8):
        rank_of_head, flops = sharding.shard_heads(wl, n)
        assert sorted(h for r in range(n) for h in sharding.heads_of_rank(rank_of_head, r)) == list(range(wl.heads))
        assert flops.max() >= flops.sum() / n
        if n <= 4:
            assert flops.max() <= 1.34 * flops.sum() / n  # five full heads dominate: 2/1, 2/1/1/1 split
    local = sharding.local_workload(wl, sharding.heads_of_rank(sharding.shard_heads(wl, 2)[0], 1))
    assert local.heads == len(local.routes) and local.grid == wl.grid


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        _rank_body(rank, world, q)
    except Exception as e:  # report instead of leaving the parent to time out
        q.put((rank, False, [repr(e)]))
        raise
    finally:
        dist.destroy_process_group()


def _rank_body(rank, world, q):
    if True:
        wl = Workload("g", (2, 4, 6), 5, 64, (1, 2, 2), (3, 3, 3), 0.5, (0, 1, 2, 1, 0), 9, False, 2)
        Q, K, V = workloads.make_qkv(wl, "cpu")
        layer = sharding.HeadShardedLayer(wl, rank, world)
        # stand-in for the rank's kernels: the oracle on the rank's heads
        def attend(b, h, route):
            q64, k64, v64 = (t[b, h].double().numpy() for t in (Q, K, V))
            if route == 0:
                return oracle.attn_full(q64, k64, v64, 0.25)
            if route == 1:
                return oracle.attn_sliding(wl.grid, wl.tile, wl.window, q64, k64, v64, 0.25)
            return oracle.attn_coreset(wl.grid, wl.bucket, float(np.float32(wl.ratio)), q64, k64, v64, 0.25)[0]
        local = torch.zeros((wl.B, len(layer.heads), wl.L, wl.d), dtype=torch.float64)
        for b in range(wl.B):
            for i, h in enumerate(layer.heads):
                local[b, i] = torch.from_numpy(attend(b, h, wl.routes[h]))
        assert torch.equal(layer.take_local(Q), Q[:, layer.heads])
        full = sharding.all_gather_heads(local, layer.rank_of_head)
        want = torch.zeros((wl.B, wl.heads, wl.L, wl.d), dtype=torch.float64)
        for b in range(wl.B):
            for h in range(wl.heads):
                want[b, h] = torch.from_numpy(attend(b, h, wl.routes[h]))
        q.put((rank, bool(torch.equal(full, want)), layer.heads))


def test_two_ranks_gather_the_full_layer_over_gloo():
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for _, ok, _ in got), got
    heads = sorted(h for _, _, hs in got for h in hs)
    assert heads == [0, 1, 2, 3, 4]


@pytest.mark.gpu
def test_ranks_shares_on_one_gpu_reproduce_the_unsharded_layer_bitwise():
    """Two ranks' shares run one after the other on one GPU (independent launches, nothing
    waits on another rank): per head the bits of the one-plan layer."""
    routes = (0, 1, 2, 1, 2, 1, 0)
    wl = Workload("shard-gpu", (6, 10, 12), len(routes), 128, (2, 4, 4), (3, 3, 3), 0.5, routes, 33, False, 2)
    Q, K, V = workloads.make_qkv(wl, "cuda:0")
    p = vb.Plan.from_workload(wl)
    O = torch.full_like(Q, float("nan"))
    p.routed_attention(Q, K, V, O)
    assert p.device_status() == 0
    p.close()
    got = torch.full_like(Q, float("nan"))
    for rank in range(2):
        layer = sharding.HeadShardedLayer(wl, rank, 2)
        q, k, v = (layer.take_local(t) for t in (Q, K, V))
        o = torch.full_like(q, float("nan"))
        layer(q, k, v, o)
        assert layer.plan.device_status() == 0
        got[:, layer.heads] = o
        layer.close()
    assert torch.equal(got.view(torch.int16), O.view(torch.int16))
