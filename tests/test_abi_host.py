"""CPU-side checks of the C ABI: the library loads, exports what vorta.h declares,
validates arguments without launching, and its host-only plan reproduces the
geometry and the work accounting of the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2505_18809_b200 import binding as vb
from paper_2505_18809_b200 import build as vbuild
from paper_2505_18809_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    vbuild.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "vorta.h")).read()
    return sorted(set(re.findall(r"VORTA_API\s+[\w\s\*]*?\b(vorta_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 14
    L = ctypes.CDLL(vb.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(vb.EXPORTS) == names


def test_status_strings():
    assert vb.vorta_status_string(0) == "ok"
    assert "timeout" in vb.vorta_status_string(vb.VORTA_ERR_TIMEOUT) or "wait" in vb.vorta_status_string(vb.VORTA_ERR_TIMEOUT)
    assert vb.vorta_status_string(99) == "unknown status"


def host_plan(**kw):
    base = dict(B=1, heads=2, grid=(4, 8, 8), d=64, tile=(2, 4, 4), window=(3, 3, 3), ratio=0.25,
                routes=(1, 2), host_only=True)
    base.update(kw)
    return vb.Plan(**base)


@pytest.mark.parametrize("kw,status", [
    (dict(d=96), vb.VORTA_ERR_UNSUPPORTED),
    (dict(tile=(16, 16, 8)), vb.VORTA_ERR_UNSUPPORTED),        # 2 048 tokens: more than 8 boxes of 128
    (dict(tile=(1, 1, 131)), vb.VORTA_ERR_UNSUPPORTED),        # 131 tokens, prime: no equal boxes of <= 128
    (dict(tile=(1, 257, 1)), vb.VORTA_ERR_UNSUPPORTED),        # an extent over 256
    (dict(bucket=(4, 3, 3)), vb.VORTA_ERR_UNSUPPORTED),        # 36 tokens
    (dict(ratio=0.0), vb.VORTA_ERR_INVALID_ARG),
    (dict(ratio=1.5), vb.VORTA_ERR_INVALID_ARG),
    (dict(routes=(1, 3)), vb.VORTA_ERR_INVALID_ARG),
    (dict(grid=(0, 8, 8)), vb.VORTA_ERR_INVALID_ARG),
    (dict(window=(3, 0, 3)), vb.VORTA_ERR_INVALID_ARG),
    (dict(tile=(2, 0, 4)), vb.VORTA_ERR_INVALID_ARG),
    (dict(grid=(2048, 2048, 1024)), vb.VORTA_ERR_INVALID_ARG),  # L >= 2^31
    (dict(scale=-1.0), vb.VORTA_ERR_INVALID_ARG),
])
def test_plan_create_rejects_bad_descriptors(kw, status):
    with pytest.raises(vb.VortaError) as e:
        host_plan(**kw)
    assert e.value.status == status


def test_null_arguments_are_errors_not_crashes():
    L = vb.lib()
    assert L.vorta_plan_create(None, None) == vb.VORTA_ERR_INVALID_ARG
    assert L.vorta_plan_destroy(None) == vb.VORTA_ERR_INVALID_ARG
    assert L.vorta_plan_info(None, None) == vb.VORTA_ERR_INVALID_ARG
    p = host_plan()
    assert L.vorta_plan_set_routes(p.handle, None, 2) == vb.VORTA_ERR_INVALID_ARG
    with pytest.raises(vb.VortaError) as e:
        p.set_routes([0, 1, 2])          # wrong length
    assert e.value.status == vb.VORTA_ERR_INVALID_ARG
    with pytest.raises(vb.VortaError) as e:
        p.set_routes([0, 7])
    assert e.value.status == vb.VORTA_ERR_INVALID_ARG
    # a host-only plan cannot launch or read device tables
    assert L.vorta_routed_attention(p.handle, 16, 16, 16, 16, None, 0, None, 0, None) == vb.VORTA_ERR_UNSUPPORTED
    assert L.vorta_plan_block_mask(p.handle, 16) == vb.VORTA_ERR_UNSUPPORTED
    assert L.vorta_coreset_select(p.handle, 16, 1, 64, 16, 16, None) == vb.VORTA_ERR_UNSUPPORTED
    # kernel selection: ids outside the enum are refused; a plan without SMs in pairs has no pair kernel;
    # a host-only plan runs no kernel
    assert L.vorta_plan_set_kernel(None, 0) == vb.VORTA_ERR_INVALID_ARG
    for bad in (-1, 4, 99):
        assert L.vorta_plan_set_kernel(p.handle, bad) == vb.VORTA_ERR_INVALID_ARG
    for ok in (vb.VORTA_KERNEL_TCGEN05, vb.VORTA_KERNEL_SIMT, vb.VORTA_KERNEL_AUTO):
        assert L.vorta_plan_set_kernel(p.handle, ok) == vb.VORTA_OK
    assert L.vorta_plan_set_kernel(p.handle, vb.VORTA_KERNEL_PAIR) == vb.VORTA_ERR_UNSUPPORTED
    assert L.vorta_plan_kernel_in_use(p.handle) < 0 and L.vorta_plan_kernel_in_use(None) < 0
    ms = (ctypes.c_float * 2)()
    assert L.vorta_plan_attention_ms_at(p.handle, 0, ctypes.byref(ms)) == vb.VORTA_ERR_UNSUPPORTED
    assert L.vorta_plan_attention_ms_at(None, 0, ctypes.byref(ms)) == vb.VORTA_ERR_INVALID_ARG
    p.close()


@pytest.mark.parametrize("name", workloads.CONFIG_NAMES)
def test_host_plan_geometry_matches_oracle(name):
    wl = workloads.config(name)
    p = vb.Plan.from_workload(wl, host_only=True)
    info = p.info
    assert info.L == wl.L
    assert info.Lc == oracle.coreset_len(wl.grid, wl.bucket, wl.ratio)
    nt = [-(-g // t) for g, t in zip(wl.grid, wl.tile)]
    assert list(info.tiles_per_axis) == nt and info.n_tiles == nt[0] * nt[1] * nt[2]
    assert info.kv_tiles_per_q_tile == int(np.prod([min(n, 2 * (w // 2) + 1) for n, w in zip(nt, wl.window)]))
    assert (info.n_full, info.n_sliding, info.n_coreset) == tuple(wl.routes.count(r) for r in (0, 1, 2))
    # algorithmic FLOPs of the sliding branch: sum over the oracle's block mask of valid-token products
    BM = oracle.sta_block_mask(wl.grid, wl.tile, wl.window).astype(np.float64)
    valid = np.zeros(info.n_tiles)
    for tid in range(info.n_tiles):
        q = (tid // (nt[1] * nt[2]), (tid // nt[2]) % nt[1], tid % nt[2])
        valid[tid] = np.prod([min(wl.tile[a], wl.grid[a] - q[a] * wl.tile[a]) for a in range(3)])
    pairs = float(valid @ BM @ valid)
    assert info.flops_sliding_head == pytest.approx(4.0 * wl.d * pairs, rel=1e-12)
    assert info.flops_full_head == pytest.approx(4.0 * wl.d * wl.L ** 2, rel=1e-12)
    assert info.flops_coreset_head == pytest.approx(4.0 * wl.d * info.Lc ** 2, rel=1e-12)
    layer = wl.B * (info.n_full * info.flops_full_head + info.n_sliding * info.flops_sliding_head +
                    info.n_coreset * info.flops_coreset_head)
    assert info.flops_layer == pytest.approx(layer, rel=1e-12)
    p.close()


def test_layer_flops_of_the_headline_configs():
    # TFLOP per layer: Wan-1.3B-480p 2.85, HunyuanVideo-720p 53.45, Wan-14B-720p 9.27
    want = {"wan1.3b-480p": 2.85, "hunyuan-720p": 53.45, "wan14b-720p": 9.27}
    for name, tf in want.items():
        p = vb.Plan.from_workload(workloads.config(name), host_only=True)
        assert p.info.flops_layer / 1e12 == pytest.approx(tf, abs=0.01)
        p.close()


def test_set_routes_updates_accounting_and_workspace():
    wl = workloads.config("wan1.3b-480p")
    p = vb.Plan.from_workload(wl, host_only=True)
    i0 = p.info
    assert i0.workspace_bytes > 0 and i0.workspace_bytes_max >= i0.workspace_bytes
    p.set_routes([0] * wl.heads)
    i1 = p.info
    assert (i1.n_full, i1.n_sliding, i1.n_coreset) == (wl.heads, 0, 0)
    assert i1.workspace_bytes == 0
    assert i1.flops_layer == pytest.approx(wl.heads * i1.flops_full_head)
    p.set_routes([2] * wl.heads)
    assert p.info.workspace_bytes == p.info.workspace_bytes_max
    p.close()


def test_default_bucket_is_the_papers():
    a = host_plan(bucket=(0, 0, 0))
    b = host_plan(bucket=(2, 3, 2))
    assert a.info.Lc == b.info.Lc == 64 and a.info.n_buckets == b.info.n_buckets == 2 * 3 * 4
    a.close()
    b.close()


def test_joint_sequence_accounting_host_only():
    """Text tokens: FLOPs per head from the definitions (pairs attended), against the oracle's masks."""
    from paper_2505_18809_b200.workloads import Workload
    wl = Workload("j", (5, 6, 7), 3, 64, (2, 2, 3), (3, 1, 3), 0.5, (0, 1, 2), 1, False, 1, (2, 3, 2), False, 19)
    p = vb.Plan.from_workload(wl, host_only=True)
    info = p.info
    p.close()
    L, Lt, d = wl.L, wl.text, wl.d
    assert info.L == L and info.text_tokens == Lt
    assert info.flops_full_head == pytest.approx(4.0 * d * (L + Lt) ** 2, rel=1e-12)
    M = oracle.sta_token_mask(wl.grid, wl.tile, wl.window)
    pairs = float(M.sum()) + L * Lt + Lt * (L + Lt)
    assert info.flops_sliding_head == pytest.approx(4.0 * d * pairs, rel=1e-12)
    Lc = oracle.coreset_len(wl.grid, wl.bucket, float(np.float32(wl.ratio)))
    assert info.Lc == Lc
    assert info.flops_coreset_head == pytest.approx(4.0 * d * (Lc + Lt) ** 2, rel=1e-12)
    with pytest.raises(vb.VortaError):
        vb.Plan(1, 1, (2, 2, 2), 64, (1, 1, 1), (1, 1, 1), 0.5, (0,), host_only=True, text=-1)


@pytest.mark.parametrize("tile,boxes", [((4, 8, 8), 2), ((6, 9, 8), 4), ((3, 9, 8), 2), ((8, 8, 16), 8),
                                        ((2, 4, 4), 1), ((3, 8, 8), 2), ((4, 9, 8), 3)])
def test_tiles_are_cut_into_equal_boxes_of_at_most_128_tokens(tile, boxes):
    """Accepted tiles: the work list has one item per pair of boxes, so its length gives the box count away
    (host-only plans have no work list: the FLOP accounting, which does not depend on the cut, is checked)."""
    grid = tuple(2 * t for t in tile)
    p = vb.Plan(1, 1, grid, 64, tile, (3, 3, 3), 0.5, (1,), host_only=True)
    info = p.info
    p.close()
    M = oracle.sta_token_mask(grid, tile, (3, 3, 3)) if grid[0] * grid[1] * grid[2] <= 4096 else None
    if M is not None:
        assert info.flops_sliding_head == pytest.approx(4.0 * 64 * float(M.sum()), rel=1e-12)
    assert tile[0] * tile[1] * tile[2] <= boxes * 128
