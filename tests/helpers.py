"""Shared helpers of the GPU parity tests: the oracle's answer for chosen rows of a
head, row sampling, and the comparison against the tolerance of the benchmark spec."""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle

MAX_ABS_TOL = 2e-2   # bf16 in, fp32 accumulate: bound on the worst element
MEAN_ABS_TOL = 2e-3  # ... and on the mean absolute error


def head_f64(x: torch.Tensor, b: int, h: int) -> np.ndarray:
    """[B, heads, L, d] bf16 (any device) -> float64 numpy [L, d] of one head."""
    return x[b, h].detach().to("cpu", torch.float64).numpy()


def oracle_head_rows(wl, Q, K, V, b, h, rows, scale=None, X=None, route=None):
    """Oracle output rows of head (b, h) under its route; rows=None means all."""
    q, k, v = head_f64(Q, b, h), head_f64(K, b, h), head_f64(V, b, h)
    scale = 1.0 / math.sqrt(wl.d) if scale is None else scale
    route = wl.routes[h] if route is None else route
    text = getattr(wl, "text", 0)
    if route == 0:
        return oracle.attn_full(q, k, v, scale, q_rows=rows)
    if route == 1:
        return oracle.attn_sliding(wl.grid, wl.tile, wl.window, q, k, v, scale, q_rows=rows, text=text)
    x = None if X is None else X
    # the float ratio is what the library sees (the ABI carries a float)
    r = float(np.float32(wl.ratio))
    O, _, _ = oracle.attn_coreset(wl.grid, wl.bucket, r, q, k, v, scale, X=x, q_rows=rows,
                                  merge=getattr(wl, "merge", False), text=text)
    return O


def sample_rows(wl, n: int, seed: int) -> np.ndarray:
    """n query tokens: the corners of the grid, tokens of the last (possibly partial)
    tile and bucket on every axis, and uniform random ones."""
    T, H, W = wl.grid
    L = wl.L
    forced = {0, L - 1, W - 1, (H - 1) * W, (T - 1) * H * W, L // 2}
    g = np.random.default_rng(seed)
    # tokens in the high-end tile of each axis (partial tiles, shifted windows)
    for _ in range(max(4, n // 8)):
        t = T - 1 - int(g.integers(0, min(T, wl.tile[0])))
        hh = H - 1 - int(g.integers(0, min(H, wl.tile[1])))
        w = W - 1 - int(g.integers(0, min(W, wl.tile[2])))
        pick = int(g.integers(0, 3))
        tt = t if pick == 0 else int(g.integers(0, T))
        hh2 = hh if pick == 1 else int(g.integers(0, H))
        ww = w if pick == 2 else int(g.integers(0, W))
        forced.add((tt * H + hh2) * W + ww)
    text = getattr(wl, "text", 0)
    if text:  # first, last and a few random text tokens
        forced |= {L, L + text - 1} | {L + int(e) for e in g.integers(0, text, size=4)}
    rows = list(sorted(forced))[:n]
    rest = n - len(rows)
    if rest > 0:
        extra = g.choice(L + text, size=min(rest, L + text), replace=False)
        rows = sorted(set(rows) | set(int(e) for e in extra))
    return np.asarray(rows, dtype=np.int64)


def _spread(g, members: np.ndarray, k: int) -> list:
    """k members of a sorted index array, one from each of k equal stretches of it
    (all of them if there are no more than k)."""
    n = len(members)
    if n <= k:
        return [int(e) for e in members]
    edges = np.linspace(0, n, k + 1).astype(np.int64)
    return [int(members[int(g.integers(edges[i], max(edges[i] + 1, edges[i + 1])))]) for i in range(k)]


def stratified_rows(wl, route: int, n: int, seed: int, core_idx=None, src_slot=None) -> np.ndarray:
    """At least ~n query rows of one head, chosen so that every unit of work of the head
    and every kind of row the route knows is hit, not merely likely to be:

    full head      every block of 128 consecutive rows (so every 256-row work item, both of
                   its query tiles, the first and the last item of the head and its short
                   tail block) gets the same number of rows;
    sliding head   every tile gets the same number of rows, spread over the tile in raster
                   order (so both boxes of a 256-token tile, every partial-tile class -- cut
                   on T, on H, on W and the corners -- and every tile whose window is shifted
                   inward at a border of any axis), plus the grid's corner tokens;
    core-set head  (core_idx, src_slot are the oracle's) every block of 128 compact rows gets
                   the same number of kept tokens, bucket centres and other kept tokens alike;
                   then as many pruned tokens, spread over the sequence, and for a share of
                   them the centre they copy, so that pruned row and centre row are both read;
    text tokens    the first, the last and a few random ones, for every route.
    """
    T, H, W = wl.grid
    L, text = wl.L, getattr(wl, "text", 0)
    g = np.random.default_rng(seed)
    rows = {0, L - 1, W - 1, (H - 1) * W, (T - 1) * H * W, L // 2}
    if route == 0:
        nblk = -(-L // 128)
        k = max(2, -(-n // nblk))
        for b in range(nblk):
            rows |= set(_spread(g, np.arange(b * 128, min(L, b * 128 + 128)), k))
    elif route == 1:
        t_, h_, w_ = wl.tile
        nt = [-(-T // t_), -(-H // h_), -(-W // w_)]
        k = max(3, -(-n // (nt[0] * nt[1] * nt[2])))
        for qt in range(nt[0]):
            for qh in range(nt[1]):
                for qw in range(nt[2]):
                    tt = np.arange(qt * t_, min(T, qt * t_ + t_))
                    hh = np.arange(qh * h_, min(H, qh * h_ + h_))
                    ww = np.arange(qw * w_, min(W, qw * w_ + w_))
                    tok = ((tt[:, None, None] * H + hh[None, :, None]) * W + ww[None, None, :]).reshape(-1)
                    rows |= set(_spread(g, tok, k))
    else:
        assert core_idx is not None and src_slot is not None
        Lc = len(core_idx)
        own = np.asarray(core_idx)[np.asarray(src_slot)] == np.arange(L)   # token kept (it is its own slot)
        nblk = -(-Lc // 128)
        k = max(2, -(-(n // 2) // nblk))
        for b in range(nblk):
            rows |= {int(core_idx[s]) for s in _spread(g, np.arange(b * 128, min(Lc, b * 128 + 128)), k)}
        pruned = np.flatnonzero(~own)
        if len(pruned):
            take = _spread(g, pruned, max(4, n // 2))
            rows |= set(take)
            rows |= {int(core_idx[src_slot[i]]) for i in take[::4]}        # the centres some of them copy
        centres = np.unique(np.asarray(src_slot)[~own]) if len(pruned) else np.zeros(0, np.int64)
        is_centre = np.zeros(Lc, bool)
        is_centre[centres] = True
        got = np.asarray(sorted(rows))
        slots = np.asarray(src_slot)[got]
        kinds = {"centre": bool((own[got] & is_centre[slots]).any()) or not len(pruned),
                 "kept non-centre": bool((own[got] & ~is_centre[slots]).any()) or bool(is_centre.all()),
                 "pruned": bool((~own[got]).any()) or not len(pruned)}
        assert all(kinds.values()), kinds
    if text:
        rows |= {L, L + text - 1} | {L + int(e) for e in g.integers(0, text, size=6)}
    return np.asarray(sorted(rows), dtype=np.int64)


def assert_close(got_rows: torch.Tensor, want: np.ndarray, what: str, stats: dict = None):
    """The parity bars of the task, per call (one head).  stats, if given, collects the worst
    absolute and RELATIVE figures seen (max-abs / max |O| and mean-abs / mean |O| of the head's
    rows): the bars are absolute, the relative figures say how much of the signal they are."""
    got = got_rows.detach().to("cpu", torch.float64).numpy()
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS_TOL, f"{what}: max-abs {err.max():.3e} > {MAX_ABS_TOL}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean-abs {err.mean():.3e} > {MEAN_ABS_TOL}"
    if stats is not None:
        mag = np.abs(want)
        stats["max_abs"] = max(stats.get("max_abs", 0.0), float(err.max()))
        stats["mean_abs"] = max(stats.get("mean_abs", 0.0), float(err.mean()))
        stats["rel_max"] = max(stats.get("rel_max", 0.0), float(err.max() / max(mag.max(), 1e-30)))
        stats["rel_mean"] = max(stats.get("rel_mean", 0.0), float(err.mean() / max(mag.mean(), 1e-30)))
        stats["rows"] = stats.get("rows", 0) + got.shape[0]
    return float(err.max()), float(err.mean())
