"""Pins for the CPU oracle: it is checked against things other than itself.

Brute force written a different way (numpy, coordinate ranges instead of tile-id
distances), torch's fp64 scaled_dot_product_attention, the numbers the paper
prints (tests/golden/paper_pins.json), closed forms and invariants.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_pins.json")))


# --------------------------------------------------------------------------- helpers
def coords(grid):
    T, H, W = grid
    t, h, w = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    return np.stack([t.ravel(), h.ravel(), w.ravel()], axis=1)  # frame-major token order


def brute_mask(grid, tile, window):
    """Token mask from key *coordinate ranges*: the window of (2*half+1) tiles,
    shifted inward at the borders, turned into [lo, hi) token coordinates."""
    c = coords(grid)
    L = c.shape[0]
    M = np.ones((L, L), dtype=bool)
    for a in range(3):
        nt = -(-grid[a] // tile[a])
        half = window[a] // 2
        if nt <= 2 * half + 1:
            continue
        q = c[:, a] // tile[a]
        centre = np.clip(q, half, nt - 1 - half)
        lo = (centre - half) * tile[a]
        hi = np.minimum((centre + half + 1) * tile[a], grid[a])
        k = c[:, a]
        M &= (k[None, :] >= lo[:, None]) & (k[None, :] < hi[:, None])
    return M


def dense_attention(Q, K, V, scale, mask=None):
    S = scale * (Q @ K.T)
    if mask is not None:
        S = np.where(mask, S, -np.inf)
    S = S - S.max(axis=1, keepdims=True)
    P = np.exp(S)
    P /= P.sum(axis=1, keepdims=True)
    return P @ V, P


def brute_select(grid, bucket, r, X):
    """Bucketed selection written with numpy sorting, bucket by bucket."""
    T, H, W = grid
    tok = np.arange(T * H * W).reshape(T, H, W)
    core, src = [], np.zeros(T * H * W, dtype=np.int64)
    for bt in range(0, T, bucket[0]):
        for bh in range(0, H, bucket[1]):
            for bw in range(0, W, bucket[2]):
                blk = tok[bt:bt + bucket[0], bh:bh + bucket[1], bw:bw + bucket[2]]
                e = blk.shape
                ids = blk.ravel()
                n = ids.size
                ci = np.ravel_multi_index((e[0] // 2, e[1] // 2, e[2] // 2), e)
                xc = X[ids[ci]]
                others = np.array([l for l in range(n) if l != ci], dtype=np.int64)
                xo = X[ids[others]]
                den = np.linalg.norm(xc) * np.linalg.norm(xo, axis=1)
                cos = np.where(den > 0, (xo @ xc) / np.where(den > 0, den, 1.0), 0.0)
                keep = max(1, int(np.floor(r * n + 0.5)))
                k = n - keep
                order = np.lexsort((others, -cos))  # primary: cos descending; then index
                pruned = set(others[order[:k]].tolist())
                seg = len(core)
                core.append(ids[ci])
                src[ids[ci]] = seg
                for l in range(n):
                    if l == ci:
                        continue
                    if l in pruned:
                        src[ids[l]] = seg
                    else:
                        src[ids[l]] = len(core)
                        core.append(ids[l])
    return np.array(core, dtype=np.int64), src


def rand_qkv(L, d, seed):
    g = np.random.default_rng(seed)
    return (g.standard_normal((L, d)), g.standard_normal((L, d)), g.standard_normal((L, d)))


GRIDS = [
    # grid, tile, window (tiles)
    ((4, 8, 8), (2, 4, 4), (3, 3, 3)),      # window covers the 2x2x2 tile grid
    ((5, 7, 9), (1, 2, 2), (3, 3, 3)),      # ragged on H and W, real windows on all axes
    ((8, 6, 10), (2, 2, 2), (3, 1, 5)),     # per-axis windows: 3, 1 (own tile only), 5
    ((10, 5, 5), (2, 2, 3), (2, 3, 3)),     # even window behaves like the next odd one
]


# --------------------------------------------------------------------------- sliding tile mask
@pytest.mark.parametrize("grid,tile,window", GRIDS)
def test_token_mask_matches_coordinate_range_brute_force(grid, tile, window):
    M = oracle.sta_token_mask(grid, tile, window).astype(bool)
    assert np.array_equal(M, brute_mask(grid, tile, window))


@pytest.mark.parametrize("grid,tile,window", GRIDS)
def test_block_mask_expands_to_token_mask(grid, tile, window):
    BM = oracle.sta_block_mask(grid, tile, window)
    c = coords(grid)
    nt = [-(-g // t) for g, t in zip(grid, tile)]
    tid = ((c[:, 0] // tile[0]) * nt[1] + c[:, 1] // tile[1]) * nt[2] + c[:, 2] // tile[2]
    assert np.array_equal(BM[tid][:, tid].astype(bool), brute_mask(grid, tile, window))


@pytest.mark.parametrize("grid,tile,window", GRIDS + [((21, 30, 52), (4, 4, 4), (3, 3, 3))])
def test_block_mask_row_counts_closed_form(grid, tile, window):
    BM = oracle.sta_block_mask(grid, tile, window)
    nt = [-(-g // t) for g, t in zip(grid, tile)]
    per_row = int(np.prod([min(n, 2 * (w // 2) + 1) for n, w in zip(nt, window)]))
    assert (BM.sum(axis=1) == per_row).all()
    assert (np.diag(BM) == 1).all()  # every tile sees itself


def test_block_mask_is_not_symmetric_at_the_border():
    BM = oracle.sta_block_mask((1, 1, 8), (1, 1, 1), (1, 1, 3))
    # tile 0's window is shifted inward to tiles {0,1,2}; tile 2's window is {1,2,3}
    assert BM[0].tolist() == [1, 1, 1, 0, 0, 0, 0, 0]
    assert BM[2].tolist() == [0, 1, 1, 1, 0, 0, 0, 0]
    assert BM[7].tolist() == [0, 0, 0, 0, 0, 1, 1, 1]
    assert BM[0, 2] == 1 and BM[2, 0] == 0


def test_paper_window_18_27_24_gives_11664_keys():
    g = GOLD["sliding_window_keys"]
    grid, tile, win = g["grid"], g["tile"], g["window_tiles"]
    assert [t * w for t, w in zip(tile, win)] == g["window_tokens"]
    assert grid[0] * grid[1] * grid[2] == g["tokens"]
    BM = oracle.sta_block_mask(grid, tile, win)
    keys = BM.sum(axis=1) * (tile[0] * tile[1] * tile[2])  # the grid divides into whole tiles
    assert (keys == g["keys_per_query"]).all()
    assert abs(g["keys_per_query"] / g["tokens"] - 0.108) < 1e-12


# --------------------------------------------------------------------------- attention
@pytest.mark.parametrize("L,d", [(37, 8), (64, 16)])
def test_full_attention_vs_torch_sdpa_and_numpy(L, d):
    Q, K, V = rand_qkv(L, d, 1)
    scale = 1.0 / np.sqrt(d)
    O, P = oracle.attn_full(Q, K, V, scale, return_probs=True)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        scale=scale)[0].numpy()
    assert np.abs(O - ref).max() < 1e-12
    On, Pn = dense_attention(Q, K, V, scale)
    assert np.abs(O - On).max() < 1e-12 and np.abs(P - Pn).max() < 1e-13
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-12 and (P >= 0).all()


def test_full_attention_row_subset():
    Q, K, V = rand_qkv(50, 8, 2)
    rows = [49, 0, 7, 7, 13]
    O = oracle.attn_full(Q, K, V, 0.3)
    assert np.array_equal(oracle.attn_full(Q, K, V, 0.3, q_rows=rows), O[rows])


@pytest.mark.parametrize("grid,tile,window", GRIDS[1:])
def test_sliding_attention_vs_brute_force_and_sdpa(grid, tile, window):
    L = grid[0] * grid[1] * grid[2]
    d = 8
    Q, K, V = rand_qkv(L, d, 3)
    scale = 1.0 / np.sqrt(d)
    O, P = oracle.attn_sliding(grid, tile, window, Q, K, V, scale, return_probs=True)
    M = brute_mask(grid, tile, window)
    On, Pn = dense_attention(Q, K, V, scale, M)
    assert np.abs(O - On).max() < 1e-12
    assert np.abs(P - Pn).max() < 1e-13
    assert (P[~M] == 0).all()
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-12
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
        attn_mask=torch.from_numpy(M)[None], scale=scale)[0].numpy()
    assert np.abs(O - ref).max() < 1e-12
    # the masked result really differs from full attention
    assert np.abs(O - oracle.attn_full(Q, K, V, scale)).max() > 1e-3


def test_window_covering_the_grid_is_full_attention():
    grid, tile, window = GRIDS[0]
    Q, K, V = rand_qkv(256, 16, 4)
    a = oracle.attn_sliding(grid, tile, window, Q, K, V, 0.25)
    b = oracle.attn_full(Q, K, V, 0.25)
    assert np.array_equal(a, b)


def test_scaling_v_and_permuting_keys():
    Q, K, V = rand_qkv(48, 8, 5)
    O = oracle.attn_full(Q, K, V, 0.35)
    assert np.abs(oracle.attn_full(Q, K, 3.0 * V, 0.35) - 3.0 * O).max() < 1e-12
    perm = np.random.default_rng(0).permutation(48)
    assert np.abs(oracle.attn_full(Q, K[perm], V[perm], 0.35) - O).max() < 1e-12
    # queries and keys are not interchangeable
    assert np.abs(oracle.attn_full(K, Q, V, 0.35) - O).max() > 1e-3


# --------------------------------------------------------------------------- core-set selection
def test_keep_count_rounding():
    # a grid that is one bucket: Lc = keep(n)
    for n_dims, r, want in [((2, 3, 2), 0.5, 6), ((2, 3, 2), 0.25, 3), ((1, 3, 2), 0.5, 3),
                            ((1, 3, 2), 0.25, 2), ((2, 2, 2), 0.5, 4), ((2, 2, 2), 0.25, 2),
                            ((1, 3, 3), 0.5, 5), ((1, 1, 1), 0.25, 1), ((1, 1, 2), 0.1, 1)]:
        assert oracle.coreset_len(n_dims, (2, 3, 3), r) == want, (n_dims, r)


def test_fig2_bucket_centre_and_dropped_count():
    g = GOLD["bcs_figure"]
    grid = g["bucket"]
    X = np.random.default_rng(6).standard_normal((9, 5))
    core, src = oracle.coreset_select(grid, grid, 0.5, X)
    assert core[0] == g["centre_local_index_0_based"]
    assert len(core) == g["kept"] and 9 - len(core) == g["dropped"]
    assert sorted(core[1:].tolist()) == core[1:].tolist()


def test_half_coreset_quarter_cost_and_config_lengths():
    g = GOLD["coreset_cost"]
    b = GOLD["bucket_defaults"]["bucket"]
    for grid in [(4, 6, 4), (8, 9, 10), (30, 45, 80)]:
        L = grid[0] * grid[1] * grid[2]
        Lc = oracle.coreset_len(grid, b, g["ratio"])
        assert 2 * Lc == L
        assert (Lc * Lc) / (L * L) == g["cost_fraction"]
    assert oracle.coreset_len((4, 8, 8), b, 0.25) == 64
    assert oracle.coreset_len((21, 30, 52), b, 0.5) == 16380
    assert oracle.coreset_len((33, 45, 80), b, 0.5) == 59400
    assert oracle.coreset_len((33, 45, 80), b, 0.25) == 30000
    assert oracle.coreset_len((21, 45, 80), b, 0.25) == 19200


@pytest.mark.parametrize("grid,bucket,r", [((4, 6, 4), (2, 3, 2), 0.5), ((5, 7, 5), (2, 3, 2), 0.25),
                                           ((3, 8, 8), (2, 3, 2), 0.5), ((4, 4, 4), (1, 2, 3), 0.7)])
def test_selection_vs_numpy_brute_force(grid, bucket, r):
    L = grid[0] * grid[1] * grid[2]
    X = np.random.default_rng(7).standard_normal((L, 12))
    core, src = oracle.coreset_select(grid, bucket, r, X)
    bc, bs = brute_select(grid, bucket, r, X)
    assert np.array_equal(core, bc) and np.array_equal(src, bs)
    assert len(core) == oracle.coreset_len(grid, bucket, r)
    # kept tokens map to themselves, every token maps to a slot of its own bucket
    assert np.array_equal(src[core], np.arange(len(core)))


def test_multiples_of_the_centre_are_pruned_before_orthogonal_tokens():
    grid = bucket = (2, 3, 2)  # one bucket of 12, centre local index (1*3+1)*2+1 = 9
    X = np.zeros((12, 4))
    X[9] = [1, 2, 0, 0]
    dup = [0, 3, 5, 10]                     # positive multiples of the centre: cos = 1
    for j, l in enumerate(dup):
        X[l] = (j + 1) * X[9]
    for l in range(12):
        if l != 9 and l not in dup:
            X[l] = [0, 0, 1 + l, 0.5]       # orthogonal to the centre: cos = 0
    core, src = oracle.coreset_select(grid, bucket, 8 / 12, X)  # keep 8, prune 4
    assert set(range(12)) - set(core.tolist()) == set(dup)
    assert core[0] == 9 and (src[dup] == 0).all()
    # negative multiples (cos = -1) are the last to go
    X[3] = -X[9]
    core, _ = oracle.coreset_select(grid, bucket, 8 / 12, X)
    assert 3 in core.tolist()


def test_ties_prune_lower_local_index_first_and_zero_norm_scores_zero():
    grid = bucket = (2, 3, 2)
    X = np.ones((12, 3))                    # all cosines equal
    core, src = oracle.coreset_select(grid, bucket, 0.5, X)
    assert core.tolist() == [9, 6, 7, 8, 10, 11]
    assert src.tolist() == [0, 0, 0, 0, 0, 0, 1, 2, 3, 0, 4, 5]
    X = np.zeros((12, 3))                   # zero norms: every score is 0, same tie-break
    core2, _ = oracle.coreset_select(grid, bucket, 0.5, X)
    assert core2.tolist() == core.tolist()


def test_ratio_one_keeps_everything_and_equals_full_attention():
    grid, bucket = (3, 5, 4), (2, 3, 2)
    L = 60
    Q, K, V = rand_qkv(L, 8, 8)
    core, src = oracle.coreset_select(grid, bucket, 1.0, K)
    assert sorted(core.tolist()) == list(range(L))
    assert np.array_equal(core[src], np.arange(L))          # src_slot inverts core_idx
    O, _, _ = oracle.attn_coreset(grid, bucket, 1.0, Q, K, V, 0.35)
    assert np.abs(O - oracle.attn_full(Q, K, V, 0.35)).max() < 1e-12


def test_coreset_attention_vs_explicit_gather_and_scatter():
    grid, bucket, r = (4, 6, 6), (2, 3, 2), 0.5
    L, d = 144, 8
    Q, K, V = rand_qkv(L, d, 9)
    X = np.random.default_rng(10).standard_normal((L, 6))
    O, core, src = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, X=X)
    bc, bs = brute_select(grid, bucket, r, X)
    assert np.array_equal(core, bc) and np.array_equal(src, bs)
    Oc, _ = dense_attention(Q[bc], K[bc], V[bc], 0.35)
    assert np.abs(O - Oc[bs]).max() < 1e-12
    # a pruned token's row is a bit-identical copy of its centre's row
    pruned = np.setdiff1d(np.arange(L), core)
    assert len(pruned) == L - len(core) > 0
    assert np.array_equal(O[pruned], O[core[src[pruned]]])
    # row subset agrees with the full call; default X is K
    rows = [143, 5, 5, 77]
    Osub, _, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, X=X, q_rows=rows)
    assert np.array_equal(Osub, O[rows])
    Ok, corek, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35)
    assert np.array_equal(corek, oracle.coreset_select(grid, bucket, r, K)[0])


def test_bucket_constant_features_make_coreset_equal_full():
    grid, bucket = (4, 6, 4), (2, 3, 2)     # divides into 8 whole buckets of 12
    g = np.random.default_rng(11)
    c = coords(grid)
    bid = ((c[:, 0] // 2) * 2 + c[:, 1] // 3) * 2 + c[:, 2] // 2
    Q, K, V = (g.standard_normal((8, 8))[bid] for _ in range(3))
    O, core, src = oracle.attn_coreset(grid, bucket, 0.5, Q, K, V, 0.35)
    assert np.abs(O - oracle.attn_full(Q, K, V, 0.35)).max() < 1e-12
    # all cosines tie, so each bucket keeps its centre and its highest local indices
    first = core[:6].tolist()
    tok = np.arange(96).reshape(grid)[:2, :3, :2].ravel()
    assert first == [tok[9], tok[6], tok[7], tok[8], tok[10], tok[11]]


def test_min_gap_reports_near_ties():
    grid = bucket = (2, 3, 2)
    X = np.random.default_rng(12).standard_normal((12, 6))
    _, _, gap = oracle.coreset_select(grid, bucket, 0.5, X, return_gap=True)
    assert 0 < gap < 2
    _, _, gap1 = oracle.coreset_select(grid, bucket, 1.0, X, return_gap=True)
    assert gap1 == np.inf


# --------------------------------------------------------------------------- router and soft mixture
def test_inference_rule_strict_inequalities_and_ties_go_to_full():
    # Eq. 4: a branch wins only if its gate is strictly the largest; build logits from chosen gates
    cases = [((0.5, 0.3, 0.2), 0), ((0.2, 0.5, 0.3), 1), ((0.2, 0.3, 0.5), 2),
             ((0.4, 0.4, 0.2), 0), ((0.2, 0.4, 0.4), 0), ((0.4, 0.2, 0.4), 0), ((1 / 3, 1 / 3, 1 / 3), 0)]
    for gates, want in cases:
        WR = np.log(np.array(gates))[None, None, :]          # one head, d_model = 1, T = 1
        g, r = oracle.router_gates(np.ones(1), WR)
        assert np.abs(g[0] - np.array(gates)).max() < 1e-12
        assert r[0] == want, gates


def test_router_gates_are_a_softmax():
    g = np.random.default_rng(20)
    T, WR = g.standard_normal(48), g.standard_normal((5, 48, 3))
    gates, routes = oracle.router_gates(T, WR)
    assert np.abs(gates.sum(axis=1) - 1).max() < 1e-12 and (gates > 0).all()
    logits = T @ WR
    assert np.array_equal(np.argmax(logits, axis=2 - 1), np.argmax(gates, axis=1))
    # a constant added to all three logits of a head changes nothing
    WR2 = WR + (g.standard_normal((5, 1, 1)) * np.ones((1, 48, 3))) * 0 + 0.0
    WR2[:, 0, :] += 3.0 / T[0]
    g2, r2 = oracle.router_gates(T, WR2)
    assert np.abs(g2 - gates).max() < 1e-9 and np.array_equal(r2, routes)
    # distinct logits: the rule is the arg-max, in the order (full, sliding, core-set)
    assert np.array_equal(routes, np.argmax(gates, axis=1).astype(np.uint8))


def test_soft_mixture_is_linear_in_the_gates_and_one_hot_gates_give_the_branch():
    grid, tile, window, bucket, r = (6, 6, 8), (2, 2, 2), (3, 3, 3), (2, 3, 2), 0.5
    Q, K, V = rand_qkv(288, 8, 21)
    full = oracle.attn_full(Q, K, V, 0.3)
    sld = oracle.attn_sliding(grid, tile, window, Q, K, V, 0.3)
    core, _, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.3)
    for onehot, want in [((1, 0, 0), full), ((0, 1, 0), sld), ((0, 0, 1), core)]:
        assert np.array_equal(oracle.soft_mixture(grid, tile, window, bucket, r, Q, K, V, 0.3, onehot), want)
    mix = oracle.soft_mixture(grid, tile, window, bucket, r, Q, K, V, 0.3, (0.2, 0.5, 0.3))
    assert np.abs(mix - (0.2 * full + 0.5 * sld + 0.3 * core)).max() < 1e-15
    rows = [0, 17, 287]
    assert np.array_equal(oracle.soft_mixture(grid, tile, window, bucket, r, Q, K, V, 0.3, (0.2, 0.5, 0.3),
                                              q_rows=rows), mix[rows])


# --------------------------------------------------------------------------- merge into the centre
def test_merge_with_one_survivor_per_bucket_is_average_pooling():
    # bucket (2,1,1), ratio .5: each pair of frames keeps one token holding the pair's mean,
    # i.e. average pooling over T (the AP_211 variant of Section 4.2), then nearest unpooling
    grid, d = (6, 3, 4), 8
    L = 72
    Q, K, V = rand_qkv(L, d, 30)
    O, core, src = oracle.attn_coreset(grid, (2, 1, 1), 0.5, Q, K, V, 0.35, merge=True)
    pool = lambda X: X.reshape(3, 2, 12, d).mean(axis=1).reshape(36, d)
    Op, _ = dense_attention(pool(Q), pool(K), pool(V), 0.35)
    want = np.repeat(Op.reshape(3, 1, 12, d), 2, axis=1).reshape(L, d)
    assert len(core) == 36
    assert np.abs(O - want).max() < 1e-12
    for bucket, shape in [((1, 3, 1), (6, 1, 3, 4)), ((1, 1, 2), (6, 3, 2, 2))]:
        Ob, cb, _ = oracle.attn_coreset(grid, bucket, 1 / 3 if bucket[1] == 3 else 0.5, Q, K, V, 0.35, merge=True)
        assert len(cb) == L // (3 if bucket[1] == 3 else 2)


def test_merge_changes_nothing_when_nothing_is_pruned_or_buckets_are_constant():
    grid, bucket = (4, 6, 4), (2, 3, 2)
    Q, K, V = rand_qkv(96, 8, 31)
    a, _, _ = oracle.attn_coreset(grid, bucket, 1.0, Q, K, V, 0.35, merge=True)
    b, _, _ = oracle.attn_coreset(grid, bucket, 1.0, Q, K, V, 0.35)
    assert np.array_equal(a, b)
    g = np.random.default_rng(32)
    c = coords(grid)
    bid = ((c[:, 0] // 2) * 2 + c[:, 1] // 3) * 2 + c[:, 2] // 2
    Qc, Kc, Vc = (g.standard_normal((8, 8))[bid] for _ in range(3))
    m, _, _ = oracle.attn_coreset(grid, bucket, 0.5, Qc, Kc, Vc, 0.35, merge=True)
    assert np.abs(m - oracle.attn_full(Qc, Kc, Vc, 0.35)).max() < 1e-12


def test_merge_vs_explicit_numpy():
    grid, bucket, r = (4, 6, 6), (2, 3, 2), 0.5
    L, d = 144, 8
    Q, K, V = rand_qkv(L, d, 33)
    O, core, src = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, merge=True)
    bc, bs = brute_select(grid, bucket, r, K)
    assert np.array_equal(core, bc)
    Qm, Km, Vm = Q[bc].copy(), K[bc].copy(), V[bc].copy()
    for s in range(len(bc)):
        grp = np.where(bs == s)[0]
        if len(grp) > 1:
            Qm[s], Km[s], Vm[s] = Q[grp].mean(0), K[grp].mean(0), V[grp].mean(0)
    Oc, _ = dense_attention(Qm, Km, Vm, 0.35)
    assert np.abs(O - Oc[bs]).max() < 1e-12
    plain, _, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35)
    assert np.abs(O - plain).max() > 1e-3


# --------------------------------------------------------------------------- joint sequences (video + text tokens)
def joint_mask(grid, tile, window, text):
    """[L + text, L + text] mask written out directly: the coordinate-range video mask, every
    text column allowed, every text row allowed."""
    Mv = brute_mask(grid, tile, window)
    L = Mv.shape[0]
    M = np.ones((L + text, L + text), dtype=bool)
    M[:L, :L] = Mv
    return M


@pytest.mark.parametrize("grid,tile,window,text", [((10, 4, 6), (2, 2, 2), (3, 3, 3), 5),
                                                   ((9, 5, 7), (2, 2, 3), (3, 1, 3), 1),
                                                   ((4, 4, 12), (1, 2, 4), (3, 3, 1), 17)])
def test_joint_sliding_attention_vs_explicit_mask(grid, tile, window, text):
    L = grid[0] * grid[1] * grid[2]
    Q, K, V = rand_qkv(L + text, 8, 21)
    O, P = oracle.attn_sliding(grid, tile, window, Q, K, V, 0.4, return_probs=True, text=text)
    M = joint_mask(grid, tile, window, text)
    Ob, Pb = dense_attention(Q, K, V, 0.4, M)
    assert np.abs(O - Ob).max() < 1e-12 and np.abs(P - Pb).max() < 1e-12
    # every query gives every text key some weight; outside its window a video query gives none
    assert (P[:, L:] > 0).all()
    assert (P[:L, :L][~M[:L, :L]] == 0).all() and (~M[:L, :L]).any()
    # a text query is a full-attention row
    Of = oracle.attn_full(Q, K, V, 0.4, q_rows=np.arange(L, L + text))
    assert np.abs(O[L:] - Of).max() < 1e-12
    # no text tokens: the video-only function
    O0 = oracle.attn_sliding(grid, tile, window, Q[:L], K[:L], V[:L], 0.4, text=0)
    assert np.array_equal(O0, oracle.attn_sliding(grid, tile, window, Q[:L], K[:L], V[:L], 0.4))
    # row subsets, text rows included
    rows = [L + text - 1, 0, L, L - 1]
    assert np.array_equal(oracle.attn_sliding(grid, tile, window, Q, K, V, 0.4, q_rows=rows, text=text), O[rows])


def test_joint_window_covering_the_grid_is_full_attention_over_all_tokens():
    grid, text = (3, 4, 5), 7
    L = 60
    Q, K, V = rand_qkv(L + text, 8, 22)
    O = oracle.attn_sliding(grid, (1, 2, 2), (3, 3, 3), Q, K, V, 0.3, text=text)
    assert np.abs(O - oracle.attn_full(Q, K, V, 0.3)).max() < 1e-12


def test_joint_coreset_keeps_every_text_token_and_prunes_video_only():
    grid, bucket, r, text = (4, 6, 6), (2, 3, 2), 0.5, 9
    L, d = 144, 8
    Q, K, V = rand_qkv(L + text, d, 23)
    O, core, src = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, text=text)
    # selection saw the video rows of K only
    bc, bs = brute_select(grid, bucket, r, K[:L])
    assert np.array_equal(core, bc) and np.array_equal(src, bs)
    # explicit pool / attend / unpool: kept video tokens, then the text tokens
    keep = np.concatenate([bc, np.arange(L, L + text)])
    Oc, _ = dense_attention(Q[keep], K[keep], V[keep], 0.35)
    assert np.abs(O[:L] - Oc[bs]).max() < 1e-12
    assert np.abs(O[L:] - Oc[len(bc):]).max() < 1e-12
    pruned = np.setdiff1d(np.arange(L), core)
    assert np.array_equal(O[pruned], O[core[src[pruned]]])
    # ratio 1: nothing pruned, so full attention over all tokens (a permutation of the keys)
    O1, _, _ = oracle.attn_coreset(grid, bucket, 1.0, Q, K, V, 0.35, text=text)
    assert np.abs(O1 - oracle.attn_full(Q, K, V, 0.35)).max() < 1e-12
    # an X of its own, with or without rows for the text tokens
    X = np.random.default_rng(24).standard_normal((L + text, 5))
    Oa, ca, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, X=X, text=text)
    Ob, cb, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, X=X[:L], text=text)
    assert np.array_equal(ca, cb) and np.array_equal(Oa, Ob)
    # merge averages video rows only: text rows of the compact sequences are untouched
    Om, _, _ = oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.35, text=text, merge=True)
    Qm, Km, Vm = Q.copy(), K.copy(), V.copy()
    for s_, c_ in enumerate(bc):
        mem = [c_] + [i for i in pruned if bs[i] == s_]
        for A, Am in ((Q, Qm), (K, Km), (V, Vm)):
            Am[c_] = A[mem].mean(axis=0)
    Ocm, _ = dense_attention(Qm[keep], Km[keep], Vm[keep], 0.35)
    assert np.abs(Om[:L] - Ocm[bs]).max() < 1e-12 and np.abs(Om[L:] - Ocm[len(bc):]).max() < 1e-12


def test_joint_soft_mixture_one_hot_gates_give_the_joint_branches():
    grid, tile, window, bucket, r, text = (4, 6, 4), (2, 3, 2), (1, 1, 3), (2, 3, 2), 0.5, 3
    Q, K, V = rand_qkv(96 + text, 8, 25)
    want = [oracle.attn_full(Q, K, V, 0.3), oracle.attn_sliding(grid, tile, window, Q, K, V, 0.3, text=text),
            oracle.attn_coreset(grid, bucket, r, Q, K, V, 0.3, text=text)[0]]
    for b in range(3):
        gates = np.eye(3)[b]
        got = oracle.soft_mixture(grid, tile, window, bucket, r, Q, K, V, 0.3, gates, text=text)
        assert np.abs(got - want[b]).max() < 1e-15
