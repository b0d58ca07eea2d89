"""GPU parity: the CUDA library against the CPU oracle, through the C ABI.

Integer results (block masks, core-set indices, scatter maps) must be bit-exact;
attention outputs must be within max-abs 2e-2 and mean-abs 2e-3 (bf16 in, fp32
accumulate), per head."""
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import assert_close, head_f64, oracle_head_rows, sample_rows, stratified_rows
from paper_2505_18809_b200 import binding as vb
from paper_2505_18809_b200 import build as vbuild
from paper_2505_18809_b200 import workloads
from paper_2505_18809_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    vbuild.build()
    vb.lib()


def small_workloads():
    W = Workload
    return [
        # name, grid, heads, d, tile, window, ratio, routes, seed, smooth
        W("tiny-c1", (4, 8, 8), 2, 64, (2, 4, 4), (3, 3, 3), 0.25, (1, 2), 0, False),
        W("three-routes-d64", (6, 10, 12), 3, 64, (2, 4, 4), (3, 3, 3), 0.5, (0, 1, 2), 21, True),
        # 4 tiles per axis and more: real windows, ragged H and W, 256-token tiles split in two boxes
        W("ragged-256tile", (9, 21, 27), 3, 128, (4, 8, 8), (3, 3, 3), 0.5, (1, 0, 2), 22, True),
        # 64-token tiles (one box per tile), ragged on T
        W("tile64", (10, 12, 20), 4, 128, (4, 4, 4), (3, 3, 3), 0.25, (1, 1, 2, 0), 23, True),
        # tile tokens not a multiple of 16 (27 -> padded to 32 columns), window 1 and 5
        W("tile27", (7, 9, 12), 3, 128, (3, 3, 3), (1, 3, 5), 0.5, (1, 2, 1), 24, True),
        # several 256-row items per head, tail block of 73 rows, batch of 2
        W("linear-tail", (3, 17, 19), 2, 128, (1, 8, 8), (3, 3, 3), 0.75, (0, 2), 25, False, 2),
        # ratio 1: the core-set is a permutation of all tokens
        W("ratio-one", (4, 6, 8), 2, 64, (2, 3, 4), (3, 3, 3), 1.0, (2, 2), 26, False),
        # bucket other than the default, grid smaller than one tile on T
        W("bucket-133", (1, 14, 15), 2, 128, (2, 4, 4), (3, 3, 3), 0.34, (2, 1), 27, False, 1, (1, 3, 3)),
        # the largest bucket the library takes (32 tokens), cut by the grid on every axis; d = 128 and 64
        W("bucket-32", (5, 9, 10), 2, 128, (2, 4, 4), (3, 3, 3), 0.3, (2, 2), 28, True, 1, (2, 4, 4)),
        W("bucket-32-d64", (6, 6, 7), 2, 64, (2, 4, 4), (3, 3, 3), 0.6, (2, 1), 29, False, 2, (4, 2, 4)),
        # tiles cut into more than two boxes, along several axes: the 6x9x8 tile of the paper's window
        # 18x27x24 (four 3x9x4 boxes of 108 tokens), a 3x9x8 tile (odd T: cut along H and W), eight boxes
        W("tile-6x9x8", (13, 20, 18), 3, 128, (6, 9, 8), (3, 3, 3), 0.5, (1, 0, 2), 71, False),
        W("tile-3x9x8", (7, 19, 17), 2, 64, (3, 9, 8), (3, 1, 3), 0.5, (1, 1), 72, False, 2),
        W("tile-8x8x16", (9, 17, 33), 2, 128, (8, 8, 16), (1, 3, 3), 0.5, (1, 1), 73, False),
        # the attention kernel's sub-block pipeline at its shortest: window of one tile, so an item has
        # one KV block: 1 sub-block (32- and 64-token tiles), 2 (128-token tile), 4 (256-token tile)
        W("one-sub-32", (4, 8, 8), 2, 128, (2, 4, 4), (1, 1, 1), 0.5, (1, 1), 41, False),
        W("one-sub-64", (8, 8, 8), 2, 64, (4, 4, 4), (1, 1, 1), 0.5, (1, 2), 42, False),
        W("two-sub-128", (4, 8, 16), 2, 128, (2, 8, 8), (1, 1, 1), 0.5, (1, 0), 43, False),
        W("four-sub-256", (8, 8, 16), 2, 128, (4, 8, 8), (1, 1, 1), 0.5, (1, 2), 44, False),
        # odd numbers of sub-blocks (3 KV tiles of 64 tokens in a window) and a cut last tile
        W("three-sub-64", (4, 4, 11), 2, 128, (4, 4, 4), (1, 1, 3), 0.5, (1, 1), 45, False),
        # linear heads shorter than one block: 40 tokens (second sub-block all masked), 70 and 129 tokens
        W("linear-40", (2, 4, 5), 2, 128, (2, 4, 4), (3, 3, 3), 1.0, (0, 2), 46, False),
        W("linear-70", (2, 5, 7), 2, 64, (2, 4, 4), (3, 3, 3), 0.6, (0, 2), 47, False),
        W("linear-129", (1, 3, 43), 2, 128, (1, 4, 4), (3, 3, 3), 0.5, (0, 2), 48, False),
    ]


KERNELS = [vb.VORTA_KERNEL_SIMT, vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_PAIR]
KERNEL_IDS = ["simt", "tcgen05", "pair"]


def set_kernel_or_skip(plan, kernel):
    """The pair kernel takes d = 128 and boxes that halve along their slowest axis; other plans refuse it."""
    try:
        plan.set_kernel(kernel)
    except vb.VortaError as e:
        if kernel == vb.VORTA_KERNEL_PAIR and e.status == vb.VORTA_ERR_UNSUPPORTED:
            plan.close()
            pytest.skip("plan not eligible for the pair kernel")
        raise


def run_layer(plan, wl, Q, K, V, kernel):
    set_kernel_or_skip(plan, kernel)
    O = torch.full_like(Q, float("nan"))
    plan.routed_attention(Q, K, V, O)
    assert plan.device_status() == 0
    return O


# --------------------------------------------------------------------------- masks
@pytest.mark.parametrize("grid,tile,window", [
    ((4, 8, 8), (2, 4, 4), (3, 3, 3)), ((9, 21, 27), (4, 8, 8), (3, 3, 3)),
    ((7, 9, 12), (3, 3, 3), (1, 3, 5)), ((10, 5, 5), (2, 2, 3), (2, 3, 3)),
    ((21, 30, 52), (4, 4, 4), (3, 3, 3)), ((33, 45, 80), (4, 8, 8), (3, 3, 3)),
    ((21, 45, 80), (4, 8, 8), (3, 3, 3)), ((30, 45, 80), (6, 9, 8), (3, 3, 3))])
def test_block_mask_bit_exact(grid, tile, window):
    p = vb.Plan(1, 1, grid, 128, tile, window, 0.5, (1,))
    got = p.block_mask()
    want = oracle.sta_block_mask(grid, tile, window)
    assert got.dtype == np.uint8 and np.array_equal(got, want)
    p.close()


# --------------------------------------------------------------------------- selection
@pytest.mark.parametrize("wl", small_workloads(), ids=lambda w: w.name)
def test_coreset_select_bit_exact_small(wl):
    _, K, _ = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    core, src = p.coreset_select(K)
    torch.cuda.synchronize()
    r = float(np.float32(wl.ratio))
    for b in range(wl.B):
        for h in range(wl.heads):
            c, s = oracle.coreset_select(wl.grid, wl.bucket, r, head_f64(K, b, h))
            assert np.array_equal(core[b, h].cpu().numpy(), c), (b, h)
            assert np.array_equal(src[b, h].cpu().numpy(), s), (b, h)
    p.close()


def test_coreset_select_other_feature_width_and_ties():
    wl = Workload("sel", (5, 7, 6), 2, 128, (2, 4, 4), (3, 3, 3), 0.5, (2, 2), 31, True)
    p = vb.Plan.from_workload(wl)
    g = torch.Generator(device=DEV).manual_seed(5)
    X = torch.randn((1, 3, wl.L, 40), generator=g, device=DEV).to(torch.bfloat16)
    X[0, 1] = 1.0                      # every cosine ties: the index tie-break decides
    X[0, 2, ::3] = 0.0                 # zero-norm rows score 0
    core, src = p.coreset_select(X)
    for h in range(3):
        c, s = oracle.coreset_select(wl.grid, wl.bucket, 0.5, head_f64(X, 0, h))
        assert np.array_equal(core[0, h].cpu().numpy(), c), h
        assert np.array_equal(src[0, h].cpu().numpy(), s), h
    p.close()


@pytest.mark.parametrize("factor", [1e-12, 1e-20, 1e12, 1e18], ids=lambda f: f"x{f:g}")
def test_coreset_select_very_small_and_very_large_norms(factor):
    """Rows far from unit scale (d = 128, the fp32-first kernel): squared norms whose product leaves
    the fp32 range must send the bucket to the fp64 scores, not to an infinite or zero fp32 one."""
    wl = Workload("sel-scale", (5, 7, 6), 3, 128, (2, 4, 4), (3, 3, 3), 0.5, (2, 2, 2), 32, True)
    p = vb.Plan.from_workload(wl)
    _, K, _ = workloads.make_qkv(wl, DEV)
    X = K.float()
    X[0, 0] *= factor                                   # every row of the head
    X[0, 1, ::2] *= factor                              # every other row: mixed magnitudes inside a bucket
    X[0, 2, : wl.L // 2] *= factor
    X[0, 2, wl.L // 2:] /= factor
    X = X.to(torch.bfloat16).contiguous()
    assert bool(torch.isfinite(X.float()).all()) and float(X.float().abs().max()) > 0
    core, src = p.coreset_select(X)
    for h in range(3):
        c, s = oracle.coreset_select(wl.grid, wl.bucket, 0.5, head_f64(X, 0, h))
        assert np.array_equal(core[0, h].cpu().numpy(), c), h
        assert np.array_equal(src[0, h].cpu().numpy(), s), h
    p.close()


# --------------------------------------------------------------------------- attention, small
@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("wl", small_workloads(), ids=lambda w: w.name)
def test_routed_attention_small_all_rows(wl, kernel):
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, kernel)
    for b in range(wl.B):
        for h in range(wl.heads):
            want = oracle_head_rows(wl, Q, K, V, b, h, None)
            assert_close(O[b, h], want, f"{wl.name} b{b} h{h} route {wl.routes[h]}")
    p.close()


@pytest.mark.parametrize("d,kernel", [(64, vb.VORTA_KERNEL_TCGEN05), (128, vb.VORTA_KERNEL_TCGEN05), (128, vb.VORTA_KERNEL_PAIR)],
                         ids=["d64-tcgen05", "d128-tcgen05", "d128-pair"])
def test_many_slices_small_heads(d, kernel):
    """Batch 3 x 70 heads of 48 tokens: slice indexing of every stage (the 5th TMA coordinate,
    compact problem numbering, per-batch core-set tables) with far more heads than SMs' items; in
    the pair kernel every item has one tile (the odd CTA of a pair only loads its K/V halves)."""
    routes = tuple((h * 7 + 3) % 3 for h in range(70))
    wl = Workload("many-slices", (2, 4, 6), 70, d, (1, 2, 2), (3, 3, 3), 0.5, routes, 61, False, 3)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, kernel)
    for b in range(wl.B):
        for h in range(0, wl.heads, 3):
            for hh in (h, min(h + 1 + b, wl.heads - 1)):
                want = oracle_head_rows(wl, Q, K, V, b, hh, None)
                assert_close(O[b, hh], want, f"b{b} h{hh} route {wl.routes[hh]}")
    p.close()


@pytest.mark.parametrize("d,kernel", [(64, vb.VORTA_KERNEL_TCGEN05), (128, vb.VORTA_KERNEL_PAIR)], ids=["d64-tcgen05", "d128-pair"])
def test_the_most_slices_the_library_takes(d, kernel):
    """B * heads = 65 535 (the limit) heads of 12 tokens: the last slices of every stage."""
    heads = 65535
    routes = tuple(h % 3 for h in range(heads))
    wl = Workload("max-slices", (1, 3, 4), heads, d, (1, 2, 2), (1, 1, 1), 0.5, routes, 62, False)
    g = torch.Generator(device=DEV).manual_seed(62)
    Q, K, V = (torch.randn((1, heads, wl.L, wl.d), generator=g, device=DEV).to(torch.bfloat16) for _ in range(3))
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, kernel)
    assert bool(torch.isfinite(O.float()).all())
    for h in (0, 1, 2, 32767, 32768, 65532, 65533, 65534):
        want = oracle_head_rows(wl, Q, K, V, 0, h, None)
        assert_close(O[0, h], want, f"h{h} route {wl.routes[h]}")
    p.close()
    with pytest.raises(vb.VortaError):
        vb.Plan(2, 32768, wl.grid, 64, wl.tile, wl.window, 0.5, (0,) * 32768, host_only=True)


@pytest.mark.parametrize("grid,tile,bucket", [((1, 1, 32767), (1, 1, 64), (1, 1, 12)), ((32767, 1, 1), (4, 1, 1), (2, 1, 1))],
                         ids=["W-32767", "T-32767"])
def test_longest_axis_the_library_takes(grid, tile, bucket):
    """A grid axis of 32 767 (the limit): tile coordinates at the top of the int16 range, 8 192
    one-box tiles along T; sampled rows of every route."""
    wl = Workload("long-axis", grid, 3, 64, tile, (3, 3, 3), 0.5, (0, 1, 2), 63, False, 1, bucket)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    assert np.array_equal(p.block_mask(), oracle.sta_block_mask(wl.grid, wl.tile, wl.window))
    O = run_layer(p, wl, Q, K, V, vb.VORTA_KERNEL_TCGEN05)
    for h in range(3):
        rows = sample_rows(wl, 64, 2000 + h)
        want = oracle_head_rows(wl, Q, K, V, 0, h, rows)
        assert_close(O[0, h][torch.from_numpy(rows).to(DEV)], want, f"h{h}")
    p.close()
    with pytest.raises(vb.VortaError):
        vb.Plan(1, 1, (1, 1, 32768), 64, tile, (3, 3, 3), 0.5, (0,), host_only=True)


@pytest.mark.parametrize("kernel", [vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_PAIR], ids=["tcgen05", "pair"])
def test_pruned_rows_copy_their_centre_and_reruns_are_bitwise_equal(kernel):
    wl = small_workloads()[2]
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O1 = run_layer(p, wl, Q, K, V, kernel)
    O2 = run_layer(p, wl, Q, K, V, kernel)
    assert torch.equal(O1.view(torch.int16), O2.view(torch.int16))
    h = wl.routes.index(2)
    core, src = oracle.coreset_select(wl.grid, wl.bucket, float(np.float32(wl.ratio)), head_f64(K, 0, h))
    owner = torch.from_numpy(core[src].astype(np.int64)).to(DEV)
    assert torch.equal(O1[0, h].view(torch.int16), O1[0, h][owner].view(torch.int16))
    p.close()


def test_routes_can_change_between_steps_and_shared_selection_features():
    wl = small_workloads()[1]
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    for routes in [(2, 2, 2), (0, 0, 0), (1, 1, 1), (2, 0, 1)]:
        p.set_routes(routes)
        O = run_layer(p, wl, Q, K, V, vb.VORTA_KERNEL_TCGEN05)
        for h in range(wl.heads):
            want = oracle_head_rows(wl, Q, K, V, 0, h, None, route=routes[h])
            assert_close(O[0, h], want, f"routes {routes} h{h}")
    # one shared feature tensor for all heads (selection on the block input, Hx = 1)
    p.set_routes((2, 2, 2))
    g = torch.Generator(device=DEV).manual_seed(9)
    X = torch.randn((1, 1, wl.L, wl.d), generator=g, device=DEV).to(torch.bfloat16)
    O = torch.empty_like(Q)
    p.routed_attention(Q, K, V, O, X=X)
    assert p.device_status() == 0
    for h in range(wl.heads):
        want = oracle_head_rows(wl, Q, K, V, 0, h, None, route=2, X=head_f64(X, 0, 0))
        assert_close(O[0, h], want, f"shared X h{h}")
    p.close()


def test_routes_alternate_between_steps_without_waiting_for_the_device():
    """The router decides per timestep (Section 3.3, Eq. 4): two route vectors taken in turn over six
    steps, each step enqueued while the one before may still be running (no synchronisation between
    set_routes and the calls), then a third, fourth, fifth and sixth vector so that kept lists are
    replaced.  Every step's output must be the oracle's for the routes it ran with, and switching back
    to a known vector must not cost a rebuild."""
    import time
    wl = Workload("alt", (6, 16, 16), 4, 128, (2, 8, 8), (3, 3, 3), 0.5, (0, 1, 2, 1), 66, False)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    ws = p.workspace(DEV) if p.info.workspace_bytes_max else None
    ws = torch.empty(int(p.info.workspace_bytes_max) + 256, dtype=torch.uint8, device=DEV)
    vectors = [(0, 1, 2, 1), (2, 2, 1, 0)]
    outs = []
    for step in range(6):
        routes = vectors[step % 2]
        p.set_routes(routes)
        O = torch.full_like(Q, float("nan"))
        p.routed_attention(Q, K, V, O, workspace=ws)
        outs.append((routes, O))
    for routes in [(1, 1, 1, 1), (0, 0, 2, 2), (2, 1, 0, 0), (1, 2, 2, 2), vectors[0]]:
        p.set_routes(routes)
        O = torch.full_like(Q, float("nan"))
        p.routed_attention(Q, K, V, O, workspace=ws)
        outs.append((routes, O))
    assert p.device_status() == 0
    want = {}
    for routes, O in outs:
        for h in range(wl.heads):
            key = (h, routes[h])
            if key not in want:
                want[key] = oracle_head_rows(wl, Q, K, V, 0, h, None, route=routes[h])
            assert_close(O[0, h], want[key], f"routes {routes} h{h}")
    # a vector whose lists are kept: no rebuild, no copy, no wait
    p.set_routes(vectors[1])
    p.set_routes(vectors[0])
    t0 = time.perf_counter()
    for _ in range(20):
        p.set_routes(vectors[1])
        p.set_routes(vectors[0])
    per_call = (time.perf_counter() - t0) / 40
    assert per_call < 0.5e-3, per_call      # measured: a few microseconds
    p.close()


def test_default_kernel_choice_follows_the_routes():
    """VORTA_KERNEL_AUTO: the pair kernel where full and core-set heads hold at least 60 % of the
    work, the single-CTA kernel otherwise; the choice is remade when the routes change."""
    wl = Workload("auto", (6, 16, 16), 3, 128, (2, 8, 8), (3, 3, 3), 0.5, (0, 1, 2), 64, False)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    for routes, want_kernel in [((0, 1, 0), vb.VORTA_KERNEL_PAIR), ((1, 1, 1), vb.VORTA_KERNEL_TCGEN05),
                                ((2, 2, 0), vb.VORTA_KERNEL_PAIR), ((1, 1, 2), vb.VORTA_KERNEL_TCGEN05),
                                ((0, 1, 2), None)]:   # near the boundary: either choice
        p.set_routes(routes)
        if want_kernel is None:
            want_kernel = p.kernel_in_use()
        assert p.kernel_in_use() == want_kernel, routes
        O = torch.full_like(Q, float("nan"))
        p.routed_attention(Q, K, V, O)
        assert p.device_status() == 0
        assert p.last_launches() == (2 if want_kernel == vb.VORTA_KERNEL_PAIR and 1 in routes else 1) + (3 if 2 in routes else 0)
        for h in range(wl.heads):
            want = oracle_head_rows(wl, Q, K, V, 0, h, None, route=routes[h])
            assert_close(O[0, h], want, f"routes {routes} h{h}")
    p.set_kernel(vb.VORTA_KERNEL_TCGEN05)
    assert p.kernel_in_use() == vb.VORTA_KERNEL_TCGEN05
    p.close()
    # d = 64: the pair kernel is refused and never chosen
    p64 = vb.Plan(1, 2, (4, 8, 8), 64, (2, 4, 4), (3, 3, 3), 0.5, (0, 0))
    assert p64.kernel_in_use() == vb.VORTA_KERNEL_TCGEN05
    with pytest.raises(vb.VortaError):
        p64.set_kernel(vb.VORTA_KERNEL_PAIR)
    p64.close()


def test_stage_times_by_launch():
    """Profiling events: the four stage times of a call, and the attention stage split by launch."""
    wl = Workload("prof", (6, 16, 16), 3, 128, (2, 8, 8), (3, 3, 3), 0.5, (0, 1, 0), 65, False)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    p.set_profiling(True)
    O = torch.empty_like(Q)
    for kernel, launches in [(vb.VORTA_KERNEL_PAIR, 2), (vb.VORTA_KERNEL_TCGEN05, 1)]:
        p.set_kernel(kernel)
        p.routed_attention(Q, K, V, O)
        torch.cuda.synchronize()
        assert p.device_status() == 0 and p.last_launches() == launches
        st, at = p.stage_ms(0), p.attention_ms(0)
        assert max(st[0], st[1], st[3]) < 0.01 < st[2]   # no core-set head: only gaps between events around the attention
        assert at[0] > 0.0 and (at[1] > 0.0) == (launches == 2)
        assert abs(at[0] + at[1] - st[2]) < 0.02 * st[2] + 1e-3
    p.close()


@pytest.mark.parametrize("kernel", [vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_PAIR], ids=["tcgen05", "pair"])
def test_growing_scores_exercise_the_lazy_rescale(kernel):
    """Keys whose norm grows along the sequence: the running maximum keeps rising, by less than
    the rescale threshold (P above 1 for a while) and by far more (O rescaled in place).  In the
    pair kernel the steps fall on blocks of all three softmax groups (shared reference maximum)."""
    wl = Workload("ramp", (4, 16, 32), 2, 128, (2, 8, 8), (3, 3, 3), 0.5, (0, 1), 41, False)
    Q, K, V = workloads.make_qkv(wl, DEV)
    ramp = torch.ones(wl.L, device=DEV)
    ramp[256:] = 2.0        # a few log2 units above the first blocks
    ramp[768:] = 4.0
    ramp[1280:] = 24.0      # tens of log2 units above everything before
    ramp[1408:] = 96.0      # and again one and two blocks later: consecutive raises by different groups
    ramp[1536:] = 400.0
    K = (K.float() * ramp[None, None, :, None]).to(torch.bfloat16).contiguous()
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, kernel)
    for h in range(wl.heads):
        want = oracle_head_rows(wl, Q, K, V, 0, h, None)
        assert_close(O[0, h], want, f"ramp h{h}")
    p.close()


def test_router_gates_and_routes_match_the_oracle():
    g = torch.Generator(device=DEV).manual_seed(60)
    heads, dm = 24, 3072
    T = torch.randn(dm, generator=g, device=DEV)
    WR = torch.randn((heads, dm, 3), generator=g, device=DEV) * 0.02
    WR[3, :, 1] = WR[3, :, 0]          # an exact tie between full and sliding
    WR[4] = 0.0                        # a three-way tie
    WR[5, :, 2] = WR[5, :, 1]          # sliding and core-set tie: neither can win, so full
    gates, routes = vb.router_gates(T, WR)
    torch.cuda.synchronize()
    want_g, want_r = oracle.router_gates(T.cpu().numpy(), WR.cpu().numpy())
    assert np.abs(gates.cpu().numpy().astype(np.float64) - want_g).max() < 1e-6
    assert np.array_equal(routes.cpu().numpy(), want_r)
    r = routes.cpu().numpy()
    assert r[4] == 0 and r[5] == 0 and r[3] in (0, 2)
    assert set(r.tolist()) == {0, 1, 2}            # the random heads spread over all three branches


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_soft_mixture_matches_the_oracle(kernel):
    wl = Workload("mix", (6, 10, 12), 3, 128, (2, 4, 4), (3, 3, 3), 0.5, (0, 1, 2), 61, False)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    set_kernel_or_skip(p, kernel)
    gates = torch.tensor([[0.2, 0.5, 0.3], [1.0, 0.0, 0.0], [0.05, 0.15, 0.8]], dtype=torch.float32, device=DEV)
    O = torch.full_like(Q, float("nan"))
    p.soft_mixture(Q, K, V, gates, O)
    assert p.device_status() == 0
    scale = 1.0 / np.sqrt(wl.d)
    for h in range(wl.heads):
        want = oracle.soft_mixture(wl.grid, wl.tile, wl.window, wl.bucket, float(np.float32(wl.ratio)),
                                   head_f64(Q, 0, h), head_f64(K, 0, h), head_f64(V, 0, h), scale,
                                   gates[h].cpu().numpy().astype(np.float64))
        assert_close(O[0, h], want, f"mixture h{h}")
    # the plan's own routes still work afterwards (the two work lists are separate)
    O2 = run_layer(p, wl, Q, K, V, kernel)
    for h in range(wl.heads):
        assert_close(O2[0, h], oracle_head_rows(wl, Q, K, V, 0, h, None), f"routed after mixture h{h}")
    p.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("bucket,ratio", [((2, 3, 2), 0.5), ((2, 1, 1), 0.5), ((1, 2, 1), 0.5), ((1, 1, 2), 0.5),
                                          ((2, 3, 2), 0.25)])
def test_merge_into_centre_and_average_pool_variants(bucket, ratio, kernel):
    # ragged grid on every axis for the (2,3,2) bucket; with one survivor per bucket the merge is average pooling
    wl = Workload("merge", (5, 10, 9), 2, 128, (2, 4, 4), (3, 3, 3), ratio, (2, 2), 70, False, 1, bucket, True)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, kernel)
    for h in range(wl.heads):
        assert_close(O[0, h], oracle_head_rows(wl, Q, K, V, 0, h, None), f"merge {bucket} h{h}")
    # without the flag the same plan gives the unmerged result, which differs
    plain = Workload("plain", wl.grid, wl.heads, wl.d, wl.tile, wl.window, ratio, wl.routes, 70, False, 1, bucket)
    p2 = vb.Plan.from_workload(plain)
    O2 = run_layer(p2, plain, Q, K, V, kernel)
    assert float((O2.float() - O.float()).abs().max()) > 1e-2
    p.close()
    p2.close()


def test_argument_errors_launch_nothing():
    wl = small_workloads()[1]
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = torch.zeros_like(Q)
    info = p.info
    ws = torch.empty(info.workspace_bytes + 256, dtype=torch.uint8, device=DEV)
    L = vb.lib()
    args = lambda q, w, n: (p.handle, q, K.data_ptr(), V.data_ptr(), O.data_ptr(), None, 0, w, n, None)
    assert L.vorta_routed_attention(*args(Q.data_ptr() + 2, ws.data_ptr(), ws.numel())) == vb.VORTA_ERR_ALIGNMENT
    assert L.vorta_routed_attention(*args(Q.data_ptr(), ws.data_ptr(), 16)) == vb.VORTA_ERR_WORKSPACE
    assert L.vorta_routed_attention(*args(Q.data_ptr(), None, 0)) == vb.VORTA_ERR_WORKSPACE
    assert L.vorta_routed_attention(*args(Q.data_ptr(), ws.data_ptr() + 16, ws.numel() - 16)) == vb.VORTA_ERR_ALIGNMENT
    assert L.vorta_routed_attention(*args(None, ws.data_ptr(), ws.numel())) == vb.VORTA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(O.abs().sum()) == 0.0
    p.close()


def test_host_buffer_entry_point_matches_device_path():
    wl = small_workloads()[3]
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, vb.VORTA_KERNEL_TCGEN05)
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    Oh = torch.empty_like(Qh).pin_memory()
    scratch = torch.empty(p.info.host_call_scratch_bytes, dtype=torch.uint8, device=DEV)
    p.routed_attention_host(Qh, Kh, Vh, Oh, scratch)
    assert p.device_status() == 0
    assert torch.equal(Oh.view(torch.int16), O.cpu().view(torch.int16))
    p.close()


@pytest.mark.parametrize("kernel", [vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_PAIR, vb.VORTA_KERNEL_AUTO],
                         ids=["tcgen05", "pair", "auto"])
def test_host_buffer_entry_point_many_heads_batch_and_route_change(kernel):
    """More heads than groups (several heads per group, uneven last group), a batch of two,
    two calls in a row on the same scratch, then new routes: always the device path's bits.
    (Under the default choice a group of heads may get another kernel than the whole layer would:
    the two paths then agree within the parity bars, not bit by bit.)"""
    routes = (0, 1, 2, 1, 2, 2, 1, 0, 1, 1, 2)
    wl = Workload("host-groups", (5, 9, 11), len(routes), 128, (2, 4, 4), (3, 3, 3), 0.5, routes, 31, False, 2)
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    scratch = torch.empty(p.info.host_call_scratch_bytes, dtype=torch.uint8, device=DEV)
    for step in range(3):
        if step == 2:
            routes = tuple((r + 1) % 3 for r in routes)
            p.set_routes(routes)
            wl = Workload("host-groups", wl.grid, wl.heads, wl.d, wl.tile, wl.window, wl.ratio, routes, 31, False, 2)
            scratch = torch.empty(p.info.host_call_scratch_bytes, dtype=torch.uint8, device=DEV)
        O = run_layer(p, wl, Q, K, V, kernel)
        Oh = torch.full_like(Qh, float("nan")).pin_memory()
        p.routed_attention_host(Qh, Kh, Vh, Oh, scratch)
        assert p.device_status() == 0
        if kernel == vb.VORTA_KERNEL_AUTO:
            for b in range(wl.B):
                for h in range(wl.heads):
                    assert_close(Oh[b, h], oracle_head_rows(wl, Q, K, V, b, h, None), f"step {step} b{b} h{h}")
        else:
            assert torch.equal(Oh.view(torch.int16), O.cpu().view(torch.int16)), step
    p.close()


# --------------------------------------------------------------------------- joint sequences (video + text tokens)
def joint_workloads():
    W = Workload
    #  name, grid, heads, d, tile, window, ratio, routes, seed, smooth, B, bucket, merge, text
    return [
        # 256-token tiles, real windows, ragged H and W; 77 text tokens (one cut text block per item)
        W("joint-256tile", (9, 21, 27), 3, 128, (4, 8, 8), (3, 3, 3), 0.5, (1, 0, 2), 51, True, 1, (2, 3, 2), False, 77),
        # 64-token tiles: text keys in blocks of 64, 130 of them (three blocks, the last of 2); batch of 2
        W("joint-tile64", (10, 12, 20), 4, 128, (4, 4, 4), (3, 3, 3), 0.25, (1, 1, 2, 0), 52, False, 2, (2, 3, 2), False, 130),
        # 27-token tiles (blocks of 32 columns, 27 real): one text token; d = 64
        W("joint-tile27-one-text", (7, 9, 12), 3, 64, (3, 3, 3), (1, 3, 5), 0.5, (1, 2, 1), 53, False, 1, (2, 3, 2), False, 1),
        # exactly two whole text blocks of 128; merged core-set heads
        W("joint-2x128-merge", (4, 8, 16), 3, 128, (2, 8, 8), (3, 3, 3), 0.5, (2, 1, 0), 54, False, 1, (2, 3, 2), True, 256),
        # more text tokens than video tokens
        W("joint-text-heavy", (2, 4, 6), 3, 128, (1, 2, 2), (1, 1, 3), 0.5, (0, 1, 2), 55, False, 1, (2, 3, 2), False, 300),
    ]


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("wl", joint_workloads(), ids=lambda w: w.name)
def test_joint_sequence_all_rows(wl, kernel):
    """Video tokens followed by text tokens: text keys visible to every query, text queries see
    every key, core-set selection prunes video tokens only."""
    Q, K, V = workloads.make_qkv(wl, DEV)
    assert Q.shape[2] == wl.L + wl.text
    p = vb.Plan.from_workload(wl)
    assert p.info.text_tokens == wl.text
    core_heads = [h for h in range(wl.heads) if wl.routes[h] == 2]
    if core_heads:
        core, src = p.coreset_select(K)
        r = float(np.float32(wl.ratio))
        for h in core_heads:
            c, s_ = oracle.coreset_select(wl.grid, wl.bucket, r, head_f64(K, 0, h)[: wl.L])
            assert np.array_equal(core[0, h].cpu().numpy(), c) and np.array_equal(src[0, h].cpu().numpy(), s_)
    O = run_layer(p, wl, Q, K, V, kernel)
    for b in range(wl.B):
        for h in range(wl.heads):
            want = oracle_head_rows(wl, Q, K, V, b, h, None)
            assert_close(O[b, h], want, f"{wl.name} b{b} h{h} route {wl.routes[h]}")
    p.close()


def test_joint_sequence_host_entry_and_soft_mixture():
    wl = joint_workloads()[0]
    Q, K, V = workloads.make_qkv(wl, DEV)
    p = vb.Plan.from_workload(wl)
    O = run_layer(p, wl, Q, K, V, vb.VORTA_KERNEL_TCGEN05)
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    Oh = torch.full_like(Qh, float("nan")).pin_memory()
    scratch = torch.empty(p.info.host_call_scratch_bytes, dtype=torch.uint8, device=DEV)
    p.routed_attention_host(Qh, Kh, Vh, Oh, scratch)
    assert p.device_status() == 0
    assert torch.equal(Oh.view(torch.int16), O.cpu().view(torch.int16))
    gates = torch.tensor([[0.2, 0.5, 0.3], [1.0, 0.0, 0.0], [0.1, 0.1, 0.8]], device=DEV)
    Om = p.soft_mixture(Q, K, V, gates)
    assert p.device_status() == 0
    scale = 1.0 / np.sqrt(wl.d)
    for h in range(wl.heads):
        want = oracle.soft_mixture(wl.grid, wl.tile, wl.window, wl.bucket, float(np.float32(wl.ratio)),
                                   head_f64(Q, 0, h), head_f64(K, 0, h), head_f64(V, 0, h), scale,
                                   gates[h].double().cpu().numpy(), text=wl.text)
        assert_close(Om[0, h], want, f"mixture h{h}")
    p.close()


# --------------------------------------------------------------------------- the named configurations
# Rows per head checked on the configurations too large for the oracle to do in full.  Every
# work item of every head is hit (helpers.stratified_rows); an environment variable lowers the
# count for a quick look, the default is what the parity claim rests on.
ROWS_PER_HEAD = int(os.environ.get("VORTA_PARITY_ROWS", "4096"))


def check_config(wl, rows_per_head, kernels=(vb.VORTA_KERNEL_AUTO, vb.VORTA_KERNEL_TCGEN05), expect_in_use=None,
                 qkv=None):
    """A whole configuration: integer stages in full, outputs on all rows or on stratified rows
    of every head, for the default kernel choice (what bench.py times) and for the kernels named."""
    Q, K, V = workloads.make_qkv(wl, DEV) if qkv is None else qkv
    p = vb.Plan.from_workload(wl)
    if expect_in_use is not None:
        assert p.kernel_in_use() == expect_in_use
    # integer stages in full: block mask, indices and scatter map of every core-set head
    assert np.array_equal(p.block_mask(), oracle.sta_block_mask(wl.grid, wl.tile, wl.window))
    core_heads = [h for h in range(wl.heads) if wl.routes[h] == 2]
    sel = {}
    if core_heads:
        core, src = p.coreset_select(K)
        for h in core_heads:
            c, s = oracle.coreset_select(wl.grid, wl.bucket, float(np.float32(wl.ratio)), head_f64(K, 0, h)[: wl.L])
            assert np.array_equal(core[0, h].cpu().numpy(), c), h
            assert np.array_equal(src[0, h].cpu().numpy(), s), h
            sel[h] = (c, s)
        del core, src
    outs = []
    for kernel in kernels:
        O = run_layer(p, wl, Q, K, V, kernel)
        assert bool(torch.isfinite(O.float()).all())
        outs.append(O)
    stats = [[{}, {}, {}] for _ in kernels]   # per kernel, per route
    for h in range(wl.heads):
        route = wl.routes[h]
        rows = None
        if rows_per_head is not None:
            c, s = sel.get(h, (None, None))
            rows = stratified_rows(wl, route, rows_per_head, 1000 + h, c, s)
            assert len(rows) >= min(rows_per_head, wl.L)
        want = oracle_head_rows(wl, Q, K, V, 0, h, rows)
        for i, (kernel, O) in enumerate(zip(kernels, outs)):
            got = O[0, h] if rows is None else O[0, h][torch.from_numpy(rows).to(DEV)]
            assert_close(got, want, f"{wl.name} h{h} route {route} kernel {kernel}", stats[i][route])
    for kernel, st in zip(kernels, stats):
        for route, s_ in enumerate(st):
            if s_:
                print(f"{wl.name} kernel {kernel} route {route}: {s_['rows']} rows, worst head max-abs {s_['max_abs']:.3e} "
                      f"(of max |O|: {s_['rel_max']:.3e}), mean-abs {s_['mean_abs']:.3e} (of mean |O|: {s_['rel_mean']:.3e})")
    p.close()


def test_config_tiny_all_rows():
    check_config(workloads.config("tiny"), None, (vb.VORTA_KERNEL_AUTO, vb.VORTA_KERNEL_SIMT, vb.VORTA_KERNEL_TCGEN05),
                 expect_in_use=vb.VORTA_KERNEL_TCGEN05)  # d = 64: the pair kernel does not apply


def test_config_wan13b_480p_all_rows():
    check_config(workloads.config("wan1.3b-480p"), None, (vb.VORTA_KERNEL_AUTO, vb.VORTA_KERNEL_SIMT, vb.VORTA_KERNEL_TCGEN05),
                 expect_in_use=vb.VORTA_KERNEL_PAIR)


def test_config_hunyuan_720p_stratified_rows():
    check_config(workloads.config("hunyuan-720p"), ROWS_PER_HEAD, expect_in_use=vb.VORTA_KERNEL_PAIR)


def test_config_wan14b_720p_stratified_rows():
    # sliding heads hold most of the work: the single-CTA kernel alone; the pair kernel is checked too
    check_config(workloads.config("wan14b-720p"), ROWS_PER_HEAD, (vb.VORTA_KERNEL_AUTO, vb.VORTA_KERNEL_PAIR),
                 expect_in_use=vb.VORTA_KERNEL_TCGEN05)


def test_config_paper_window_18x27x24_stratified_rows():
    check_config(workloads.config("hunyuan-30x45x80-tile6x9x8"), ROWS_PER_HEAD // 4)


def test_config_hunyuan_720p_with_256_text_tokens_stratified_rows():
    check_config(workloads.config("hunyuan-720p-text256"), ROWS_PER_HEAD // 4)


@pytest.mark.parametrize("wl", workloads.route_mix_sweep(), ids=lambda w: w.name)
def test_config_route_mix_sweep_stratified_rows(wl):
    # all eight corners of the sweep: full-head fraction 0 / .25 / .5 / 1 x core-set ratio .25 / .5
    check_config(wl, ROWS_PER_HEAD, (vb.VORTA_KERNEL_AUTO,))


def test_peaked_softmax_at_the_headline_shape():
    """118 800 tokens, one head per route, keys scaled so that a few of them carry a row's mass
    (|O| is then of the size of |V| and the absolute bars bite) and so that the score level keeps
    rising along the sequence, in steps below and above the lazy-rescale threshold: every query
    row moves its reference maximum many times, in every softmax group of the pair kernel."""
    wl = workloads.config("hunyuan-720p-3h")
    Q, K, V = workloads.make_qkv(wl, DEV)
    chunk = torch.arange(wl.L, device=DEV) // 1280            # 93 stretches, not aligned with any block
    level = 4.0 * (1.0 + 0.08 * chunk.float())
    level[chunk % 11 == 10] *= 1.6                            # a few jumps far above the threshold
    K = (K.float() * level[None, None, :, None]).to(torch.bfloat16).contiguous()
    check_config(wl, ROWS_PER_HEAD, (vb.VORTA_KERNEL_AUTO, vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_PAIR), qkv=(Q, K, V))
