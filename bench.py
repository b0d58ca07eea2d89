#!/usr/bin/env python
"""Benchmark of one routed-attention layer (select + gather + attention + scatter).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
  python bench.py --sweep [--steps K]     the route-mix sweep with the speed-up over all-full attention

A step is one call of vorta_routed_attention on one layer's Q/K/V (seeded
synthetic, resident in HBM).  The line printed by rank 0 carries:
  value        effective TFLOP/s = algorithmic FLOPs of the layer / time per step
               (4*d*pairs the method attends: L^2 full, valid window pairs sliding,
               Lc^2 core-set), whole job over all ranks
  ms_per_step  ms per layer
  roofline     the attention kernel alone: algorithmic FLOPs / its CUDA-event time
               against the measured dense bf16 peak
  e2e          the same metric through vorta_routed_attention_host with pinned HOST
               buffers (H2D of Q, K, V and D2H of O inside the timed region)
  cpu_baseline the fp64 CPU oracle timed on a bounded sample of rows of the same workload
With --impl reference the oracle itself is the timed arm.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed_attention_effective_tflops"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "hunyuan-720p"
FALLBACK_PEAK_TFLOPS = 1590.0   # used only if MEASURED_PEAKS.json is absent
# DRAM traffic of the attention kernels per algorithmic byte, from ncu captures of the three-head
# profiling case (profiles/): the single-CTA kernel over all three heads read 441.5 MB and wrote 62.6 MB
# for 304.1 MB of algorithmic bytes; the pair kernel over the full and the core-set head read 445.8 MB
# and wrote 68.5 MB for 182.5 MB.  A launch of another workload is estimated by the same ratio.
ATTENTION_TRAFFIC_PER_ALGORITHMIC_BYTE = 504.1 / 304.1
PAIR_KERNEL_TRAFFIC_PER_ALGORITHMIC_BYTE = 514.3 / 182.5
# VORTA_KERNEL_* id -> what the attention stage launches
ATTENTION_KERNEL_NAMES = {
    0: "attention_sm100_kernel",
    2: "attention_sm100_pair_kernel (full and core-set heads) then attention_sm100_kernel (sliding heads)",
    1: "attention_simt_kernel",
}


def attention_algorithmic_bytes(info, wl) -> float:
    """Q, K, V read and O written once per full or sliding head; the gathered Q, K, V, O per core-set head."""
    row = wl.d * 2
    return wl.B * ((info.n_full + info.n_sliding) * 4.0 * info.L * row + info.n_coreset * 4.0 * info.Lc * row)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16": float(p["bf16_tflops"]), "bf16_sustained": float(p.get("bf16_tflops_sustained", 0.0)),
                "hbm": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16": FALLBACK_PEAK_TFLOPS, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


def get_workload(name):
    from paper_2505_18809_b200 import workloads
    if name in workloads.CONFIG_NAMES or name in workloads.PROFILE_NAMES or name in workloads.JOINT_NAMES:
        return workloads.config(name)
    for w in workloads.route_mix_sweep():
        if w.name == name:
            return w
    raise SystemExit(f"unknown workload {name}")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), line.strip()))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()   # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        for ts, line in self.rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                clk, mx = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            smax = mx
            if t0 - 0.1 <= ts <= t1 + 0.3:
                sm.append(clk)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:
            sm = [float(l.split(",")[0]) for _, l in self.rows[-3:] if l and l.split(",")[0].strip().replace(".", "").isdigit()]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- oracle timing
def _window_keys(wl, token: int) -> int:
    """Number of keys Algorithm 1 lets this query see (for the FLOP count of a sampled row)."""
    T, H, W = wl.grid
    c = (token // (H * W), (token // W) % H, token % W)
    n = 1
    for a in range(3):
        nt = -(-wl.grid[a] // wl.tile[a])
        half = wl.window[a] // 2
        if nt <= 2 * half + 1:
            n *= wl.grid[a]
            continue
        q = c[a] // wl.tile[a]
        centre = min(max(q, half), nt - 1 - half)
        lo, hi = (centre - half) * wl.tile[a], min((centre + half + 1) * wl.tile[a], wl.grid[a])
        n *= hi - lo
    return n


def time_oracle(wl, Q, K, V, rows_per_head: int, budget_s: float, seed: int = 0):
    import numpy as np
    import torch
    import oracle
    scale = 1.0 / math.sqrt(wl.d)
    Lc = oracle.coreset_len(wl.grid, wl.bucket, float(np.float32(wl.ratio)))
    g = np.random.default_rng(seed)
    flops, t_total, heads_done = 0.0, 0.0, 0
    text = getattr(wl, "text", 0)
    n_rows = wl.L + text
    for h in range(wl.heads):
        if t_total > budget_s:
            break
        q, k, v = (x[0, h].to("cpu", torch.float64).numpy() for x in (Q, K, V))
        rows = np.sort(g.choice(n_rows, size=min(rows_per_head, n_rows), replace=False)).astype(np.int64)
        t0 = time.perf_counter()
        if wl.routes[h] == 0:
            oracle.attn_full(q, k, v, scale, q_rows=rows)
            f = 4.0 * wl.d * n_rows * len(rows)
        elif wl.routes[h] == 1:
            oracle.attn_sliding(wl.grid, wl.tile, wl.window, q, k, v, scale, q_rows=rows, text=text)
            # a video query: its window and every text key; a text query: every key
            f = 4.0 * wl.d * sum(_window_keys(wl, int(r)) + text if r < wl.L else n_rows for r in rows)
        else:
            _, _, src = oracle.attn_coreset(wl.grid, wl.bucket, float(np.float32(wl.ratio)), q, k, v, scale,
                                            q_rows=rows, text=text)
            slots = set(src[rows[rows < wl.L]].tolist()) | set((Lc + (rows[rows >= wl.L] - wl.L)).tolist())
            f = 4.0 * wl.d * (Lc + text) * len(slots)
        t_total += time.perf_counter() - t0
        flops += f
        heads_done += 1
    return flops, t_total, heads_done, oracle.num_threads()


# ----------------------------------------------------------------------------- multi-rank aggregation
def reduce_max_ms(ms_local: float, world: int, device) -> float:
    """The job's time is the slowest rank's: max-reduce over the process group (if any)."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank_step: float, world: int, ms_per_step: float) -> float:
    """Every rank runs its own layer (heads are independent, nothing is exchanged): the job's
    throughput is the work of all ranks over the slowest rank's time."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def config_dict(wl, info, n_bytes_per_tensor: float, shard_heads: bool = False, mixture: bool = False):
    """The `config` object of the JSON line: the same for the library's arm and the oracle's."""
    return {"workload": wl.name + ("+soft-mixture" if mixture else ""), "grid": list(wl.grid),
            "tokens": wl.L, "text_tokens": getattr(wl, "text", 0), "heads": wl.heads,
            "d": wl.d, "tile": list(wl.tile), "window_tiles": list(wl.window),
            "coreset_ratio": wl.ratio, "routes": list(wl.routes),
            "heads_full_sliding_coreset": [info.n_full, info.n_sliding, info.n_coreset],
            "algorithmic_tflop_per_layer": info.flops_layer / 1e12,
            "l2": "inputs (3 x %.0f MB) larger than L2" % (n_bytes_per_tensor / 1e6),
            "per_rank": ("heads of one layer split over the GPUs (vorta_shard_heads), no collective on the "
                         "data path; roofline and stages are rank 0's share") if shard_heads
            else "one layer per GPU, no collective on the data path"}


def sharded_job_tflops(full_layer_flops: float, ms_per_step: float) -> float:
    """--shard-heads (strong scaling): ONE layer whose heads are split over the ranks; the job's
    throughput is the whole layer's work over the slowest rank's time."""
    return full_layer_flops / (ms_per_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------- arms
def run_reference(args):
    """The oracle as the timed arm: each step is a bounded sample of rows of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2505_18809_b200 import workloads
    oracle.build()
    wl = get_workload(args.workload)
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    Q, K, V = workloads.make_qkv(wl, dev)
    Q, K, V = Q.cpu(), K.cpu(), V.cpu()
    rows = args.reference_rows
    for _ in range(args.warmup):
        time_oracle(wl, Q, K, V, max(1, rows // 4), 5.0)
    flops, secs = 0.0, 0.0
    heads = 0
    for s in range(args.steps):
        f, t, heads, threads = time_oracle(wl, Q, K, V, rows, 120.0 / max(1, args.steps), seed=s)
        flops += f
        secs += t
    value = flops / secs / 1e12
    sample = f"{rows} random query rows of each of {heads} heads per step, all their keys"
    from paper_2505_18809_b200 import binding as vb
    from paper_2505_18809_b200 import build as vbuild
    vbuild.build()
    host_plan = vb.Plan.from_workload(wl, host_only=True)   # geometry and FLOP accounting only: launches nothing
    cfg = config_dict(wl, host_plan.info, Q.numel() * 2)
    host_plan.close()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": cfg,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2505_18809_b200 import binding as vb
    from paper_2505_18809_b200 import build as vbuild
    from paper_2505_18809_b200 import workloads

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        vbuild.build()
    if world > 1:
        dist.barrier()
    vb.lib()

    wl = get_workload(args.workload)
    if args.merge:
        import dataclasses
        wl = dataclasses.replace(wl, name=wl.name + "+merge", merge=True)
    pk = peaks()
    full_layer_flops = None
    if args.shard_heads:
        # strong scaling: ONE layer, its heads split over the ranks by the library's partition
        # (head-sharded Q, K, V, no collective on the data path); every rank makes only its heads
        from paper_2505_18809_b200 import sharding
        if world > wl.heads:
            raise SystemExit("--shard-heads needs at least one head per rank")
        host_plan = vb.Plan.from_workload(wl, host_only=True)
        full_layer_flops = host_plan.info.flops_layer
        host_plan.close()
        rank_of_head, _ = sharding.shard_heads(wl, world)
        wl = sharding.local_workload(wl, sharding.heads_of_rank(rank_of_head, rank))
    # every rank holds its own layer (heads are independent: no exchange inside the op)
    Q, K, V = workloads.make_qkv(wl, dev)
    O = torch.empty_like(Q)
    plan = vb.Plan.from_workload(wl, device=local)
    info = plan.info
    ws = plan.workspace(dev)
    plan.set_profiling(True)
    if args.kernel >= 0:
        plan.set_kernel(args.kernel)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    flops_step = info.flops_layer
    if args.mixture:
        # Eq. 5: every head runs all three branches; the gates only weight the outputs
        gates = torch.softmax(torch.randn((wl.heads, 3), device=dev), dim=1).contiguous()
        mix_ws = torch.empty(int(info.mixture_workspace_bytes), dtype=torch.uint8, device=dev)
        flops_step = wl.B * wl.heads * (info.flops_full_head + info.flops_sliding_head + info.flops_coreset_head)

    def step():
        if args.mixture:
            plan.soft_mixture(Q, K, V, gates, O, workspace=mix_ws)
        else:
            plan.routed_attention(Q, K, V, O, workspace=ws)

    warmup_run = max(args.warmup, 3)   # the timing rules ask for at least three
    for _ in range(warmup_run):
        step()
    assert plan.device_status() == 0

    # ---- timed region: exactly K steps, device time, max over ranks
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]   # between the steps: median and min
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    launches = 0
    marks[0].record(stream)
    for i in range(args.steps):
        step()
        marks[i + 1].record(stream)
        launches += plan.last_launches()
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms_total = e0.elapsed_time(e1)
    per_step = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    assert plan.device_status() == 0
    ms_total = reduce_max_ms(ms_total, world, dev)
    ms_step = ms_total / args.steps
    value = whole_job_tflops(flops_step, world, ms_step)
    if full_layer_flops is not None:
        value = sharded_job_tflops(full_layer_flops, ms_step)

    # stage times of the timed steps (CUDA events recorded by the library on the same stream)
    n_hist = min(args.steps, 64)
    if args.mixture:
        plan.set_profiling(True)
        stages = [[0.0, 0.0, ms_step, 0.0]]     # the mixture call is not split into stages
        n_hist = 1
    else:
        stages = [plan.stage_ms(i) for i in range(n_hist)]
    st = [sum(s[i] for s in stages) / n_hist for i in range(4)]
    attn_ms = st[2]
    # the attention stage by launch: [pair kernel or the only kernel, single-CTA kernel after the pair kernel]
    by_launch = [attn_ms, 0.0]
    if not args.mixture:
        parts = [plan.attention_ms(i) for i in range(n_hist)]
        by_launch = [sum(x[i] for x in parts) / n_hist for i in range(2)]
    n_core = info.n_coreset * wl.B

    out = None
    if rank == 0:
        kernel_used = plan.kernel_in_use()
        stage_tflops = flops_step / (attn_ms * 1e-3) / 1e12
        row = wl.d * 2
        two = by_launch[1] > 0.0
        if two:
            # Two attention launches: the dominant kernel is the pair kernel (full and core-set heads);
            # its own FLOPs and bytes over its own time.  The whole stage is reported beside it.
            name = "attention_sm100_pair_kernel"
            k_flops = wl.B * (info.n_full * info.flops_full_head + info.n_coreset * info.flops_coreset_head)
            k_ms = by_launch[0]
            k_bytes = wl.B * (info.n_full * 4.0 * info.L * row + info.n_coreset * 4.0 * info.Lc * row)
            k_ratio = PAIR_KERNEL_TRAFFIC_PER_ALGORITHMIC_BYTE
        else:
            name = ATTENTION_KERNEL_NAMES.get(kernel_used, str(kernel_used))
            if kernel_used == 2 and not args.mixture:   # one launch: only one kind of head is present
                name = "attention_sm100_pair_kernel" if info.n_sliding == 0 else "attention_sm100_kernel"
            k_flops, k_ms, k_bytes = flops_step, attn_ms, attention_algorithmic_bytes(info, wl)
            k_ratio = (PAIR_KERNEL_TRAFFIC_PER_ALGORITHMIC_BYTE if name == "attention_sm100_pair_kernel"
                       else ATTENTION_TRAFFIC_PER_ALGORITHMIC_BYTE)
        achieved = k_flops / (k_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": name, "achieved": achieved,
                    "peak": pk["bf16"], "unit": UNIT, "frac": achieved / pk["bf16"],
                    "peak_source": f"{pk['source']} burst bf16",
                    "frac_of_sustained": achieved / pk["bf16_sustained"] if pk["bf16_sustained"] else None,
                    "frac_of_nominal_2250": achieved / 2250.0,
                    "kernel_ms": k_ms, "kernel_algorithmic_tflop": k_flops / 1e12,
                    "algorithmic_bytes": k_bytes,
                    "traffic": k_ratio * k_bytes if not args.mixture else None,
                    "traffic_source": "ncu dram bytes of this kernel in the 3-head capture, scaled by algorithmic bytes",
                    "attention_stage": {"kernels": ATTENTION_KERNEL_NAMES.get(kernel_used, str(kernel_used)),
                                        "ms_by_launch": by_launch, "ms": attn_ms, "tflops": stage_tflops,
                                        "frac": stage_tflops / pk["bf16"],
                                        "frac_of_sustained": stage_tflops / pk["bf16_sustained"] if pk["bf16_sustained"] else None,
                                        "issued_tflops": info.flops_issued_layer / (attn_ms * 1e-3) / 1e12}}
        gbs = lambda b, ms: (b / (ms * 1e-3) / 1e9) if ms > 0 else None
        stage = {"select_ms": st[0], "gather_ms": st[1], "attention_ms": st[2], "scatter_ms": st[3],
                 "select_gbs": gbs(n_core * info.select_bytes_head, st[0]),
                 "gather_gbs": gbs(n_core * info.gather_bytes_head, st[1]),
                 "scatter_gbs": gbs(n_core * info.scatter_bytes_head, st[3]),
                 "hbm_peak_gbs": pk["hbm"]}
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": warmup_run, "ms_per_step": ms_step, "ms_per_layer": ms_step,
               "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
               "higher_is_better": True, "scaling": "strong" if args.shard_heads else "weak", "vs_baseline": None,
               "dtype": "bf16",
               "data": "synthetic",
               "config": config_dict(wl, info, Q.numel() * 2, args.shard_heads, args.mixture),
               "issued_tflop_per_layer": info.flops_issued_layer / 1e12,
               "frac_of_bf16_peak": value / world / pk["bf16"],
               "roofline": roofline, "stages": stage, "gpu_launches": launches, "clocks": clocks}
        if clocks and clocks.get("sm_mhz"):
            # the run may sit on the power cap: time x clock tells a cycle win from a clock change
            out["mcycles_per_step_at_sampled_clock"] = ms_step * clocks["sm_mhz"] * 1e-3   # ms x MHz = 1e3 cycles

    # ---- end to end through the host-buffer entry point (rank-local, max over ranks)
    e2e = None
    if not args.no_e2e and not args.mixture:
        Qh, Kh, Vh = (torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in (Q, K, V))
        Oh = torch.empty(Q.shape, dtype=Q.dtype, pin_memory=True)
        scratch = torch.empty(int(info.host_call_scratch_bytes), dtype=torch.uint8, device=dev)
        for _ in range(2):
            plan.routed_attention_host(Qh, Kh, Vh, Oh, scratch)
        barrier()
        n_e2e = max(2, args.steps)
        e0.record(stream)
        for _ in range(n_e2e):
            plan.routed_attention_host(Qh, Kh, Vh, Oh, scratch)
        e1.record(stream)
        barrier()
        ms_e2e = reduce_max_ms(e0.elapsed_time(e1) / n_e2e, world, dev)
        tb = Q.numel() * 2
        e2e_value = (sharded_job_tflops(full_layer_flops, ms_e2e) if full_layer_flops is not None
                     else whole_job_tflops(info.flops_layer, world, ms_e2e))
        e2e = {"value": e2e_value, "unit": UNIT,
               "ms_per_step": ms_e2e, "steps": n_e2e, "h2d_bytes_per_step": 3 * tb, "d2h_bytes_per_step": tb,
               "api": "vorta_routed_attention_host (pinned host Q, K, V in; O out)"}
        del scratch, Qh, Kh, Vh
    if rank == 0:
        out["e2e"] = e2e

    # ---- the oracle on the host cores, rank 0 at N = 1 only
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        Qc, Kc, Vc = Q.cpu(), K.cpu(), V.cpu()
        rows = args.cpu_rows
        flops, secs, heads, threads = time_oracle(wl, Qc, Kc, Vc, rows, 25.0)
        out["cpu_baseline"] = {"value": flops / secs / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                               "seconds": secs,
                               "sample": f"{rows} random query rows of each of the first {heads} heads "
                                         f"(of {wl.heads}), all their keys; fp64"}
    elif rank == 0:
        out["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(out))
    plan.close()
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """The route-mix sweep on the HunyuanVideo-720p shape (full-head fraction 0 / .25 / .5 / 1, the rest
    split evenly between sliding and core-set, core-set ratio .25 / .5; seeds 4-11): per point ms/layer,
    effective TFLOP/s, fraction of the measured peak and the speed-up over the SAME kernels running all
    24 heads as full attention.  One GPU; prints a table and one JSON line ({"sweep": [...]})."""
    import dataclasses
    import torch
    from paper_2505_18809_b200 import binding as vb
    from paper_2505_18809_b200 import build as vbuild
    from paper_2505_18809_b200 import workloads
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(0)
    dev = "cuda:0"
    vbuild.build()
    vb.lib()
    pk = peaks()
    stream = torch.cuda.current_stream()
    points = workloads.route_mix_sweep()
    ref = dataclasses.replace(points[0], name="hunyuan-720p-all-full", routes=(0,) * points[0].heads)
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    stamps = []
    for wl in [ref] + points:
        Q, K, V = workloads.make_qkv(wl, dev)
        O = torch.empty_like(Q)
        plan = vb.Plan.from_workload(wl)
        if args.kernel >= 0:
            plan.set_kernel(args.kernel)
        info = plan.info
        ws = plan.workspace(dev)
        for _ in range(max(args.warmup, 3)):
            plan.routed_attention(Q, K, V, O, workspace=ws)
        assert plan.device_status() == 0
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        torch.cuda.synchronize()
        t0 = time.time()
        marks[0].record(stream)
        for i in range(args.steps):
            plan.routed_attention(Q, K, V, O, workspace=ws)
            marks[i + 1].record(stream)
        torch.cuda.synchronize()
        t1 = time.time()
        assert plan.device_status() == 0
        per_step = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
        ms = marks[0].elapsed_time(marks[-1]) / args.steps
        stamps.append((t0, t1))
        rows.append({"workload": wl.name, "heads_full_sliding_coreset": [info.n_full, info.n_sliding, info.n_coreset],
                     "coreset_ratio": wl.ratio, "seed": wl.seed, "algorithmic_tflop": info.flops_layer / 1e12,
                     "ms_per_layer": ms, "ms_median": statistics.median(per_step), "ms_min": min(per_step),
                     "tflops": info.flops_layer / (ms * 1e-3) / 1e12,
                     "frac_of_bf16_peak": info.flops_layer / (ms * 1e-3) / 1e12 / pk["bf16"],
                     "kernel_in_use": plan.kernel_in_use()})
        plan.close()
        del Q, K, V, O, ws
        torch.cuda.empty_cache()
    all_full_ms = rows[0]["ms_per_layer"]
    for r, (t0, t1) in zip(rows, stamps):
        r["speedup_vs_all_full"] = all_full_ms / r["ms_per_layer"]
    clocks = sampler.stop(stamps[0][0], stamps[-1][1])
    print("| workload | full/sliding/core-set | r | TFLOP | ms/layer (median, min) | TFLOP/s | of peak | speed-up vs all-full |",
          file=sys.stderr)
    print("|---|---|---|---|---|---|---|---|", file=sys.stderr)
    for r in rows:
        f, s_, c = r["heads_full_sliding_coreset"]
        print(f"| {r['workload']} | {f}/{s_}/{c} | {r['coreset_ratio']:g} | {r['algorithmic_tflop']:.2f} | "
              f"{r['ms_per_layer']:.2f} ({r['ms_median']:.2f}, {r['ms_min']:.2f}) | {r['tflops']:.0f} | "
              f"{100 * r['frac_of_bf16_peak']:.1f} % | {r['speedup_vs_all_full']:.2f}x |", file=sys.stderr)
    print(json.dumps({"metric": METRIC, "unit": UNIT, "sweep": rows, "steps": args.steps, "warmup": max(args.warmup, 3),
                      "peak": pk["bf16"], "peak_source": f"{pk['source']} burst bf16", "clocks": clocks,
                      "dtype": "bf16", "data": "synthetic"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-rows", type=int, default=800, help="oracle rows per head for cpu_baseline")
    ap.add_argument("--reference-rows", type=int, default=16, help="oracle rows per head per step (--impl reference)")
    ap.add_argument("--kernel", type=int, default=-1, help="attention kernel id (see vorta.h); -1 = library default")
    ap.add_argument("--mixture", action="store_true", help="time vorta_soft_mixture (all three branches per head)")
    ap.add_argument("--merge", action="store_true",
                    help="core-set heads merge the pruned tokens into their centre (mean) before attention")
    ap.add_argument("--shard-heads", action="store_true",
                    help="strong scaling: one layer, heads split over the ranks (default: one layer per rank)")
    ap.add_argument("--sweep", action="store_true",
                    help="the route-mix sweep on the HunyuanVideo-720p shape, with the speed-up over all-full attention")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
