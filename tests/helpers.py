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


def assert_close(got_rows: torch.Tensor, want: np.ndarray, what: str):
    got = got_rows.detach().to("cpu", torch.float64).numpy()
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS_TOL, f"{what}: max-abs {err.max():.3e} > {MAX_ABS_TOL}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean-abs {err.mean():.3e} > {MEAN_ABS_TOL}"
    return float(err.max()), float(err.mean())
