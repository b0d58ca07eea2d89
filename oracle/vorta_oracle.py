"""ctypes front end of ``vorta_oracle.c`` (TEST INFRASTRUCTURE, not product code).

Every function takes numpy arrays, converts them to contiguous float64 and calls
the C routine of the same name; see the C file for what each one computes and
which passage of the paper it follows.  ``build()`` compiles the C file with gcc
(OpenMP) into ``oracle/libvorta_oracle.so``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vorta_oracle.c")
_LIB = os.path.join(_HERE, "libvorta_oracle.so")
_lib: Optional[ctypes.CDLL] = None

_i32p = ctypes.POINTER(ctypes.c_int32)
_i64p = ctypes.POINTER(ctypes.c_int64)
_f64p = ctypes.POINTER(ctypes.c_double)
_u8p = ctypes.POINTER(ctypes.c_uint8)


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".{os.getpid()}.tmp"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden", "-std=c11",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    lib.vo_sta_token_mask.argtypes = [_i32p, _i32p, _i32p, _u8p]
    lib.vo_sta_token_mask.restype = ctypes.c_int
    lib.vo_sta_block_mask.argtypes = [_i32p, _i32p, _i32p, _u8p]
    lib.vo_sta_block_mask.restype = ctypes.c_int
    lib.vo_attn_full.argtypes = [ctypes.c_int64, ctypes.c_int32, _f64p, _f64p, _f64p,
                                 ctypes.c_double, ctypes.c_int64, _i64p, _f64p, _f64p]
    lib.vo_attn_full.restype = ctypes.c_int
    lib.vo_attn_sliding.argtypes = [_i32p, _i32p, _i32p, ctypes.c_int32, _f64p, _f64p, _f64p,
                                    ctypes.c_double, ctypes.c_int64, _i64p, _f64p, _f64p]
    lib.vo_attn_sliding.restype = ctypes.c_int
    lib.vo_attn_sliding_joint.argtypes = [_i32p, _i32p, _i32p, ctypes.c_int64, ctypes.c_int32, _f64p, _f64p,
                                          _f64p, ctypes.c_double, ctypes.c_int64, _i64p, _f64p, _f64p]
    lib.vo_attn_sliding_joint.restype = ctypes.c_int
    lib.vo_coreset_len.argtypes = [_i32p, _i32p, ctypes.c_double]
    lib.vo_coreset_len.restype = ctypes.c_int64
    lib.vo_coreset_select.argtypes = [_i32p, _i32p, ctypes.c_double, _f64p, ctypes.c_int32,
                                      _i32p, _i32p, _f64p]
    lib.vo_coreset_select.restype = ctypes.c_int64
    lib.vo_attn_coreset.argtypes = [_i32p, _i32p, ctypes.c_double, ctypes.c_int32, _f64p, _f64p,
                                    _f64p, _f64p, ctypes.c_int32, ctypes.c_double, ctypes.c_int64,
                                    _i64p, _f64p, _i32p, _i32p]
    lib.vo_attn_coreset.restype = ctypes.c_int64
    lib.vo_attn_coreset_ex.argtypes = lib.vo_attn_coreset.argtypes + [ctypes.c_int]
    lib.vo_attn_coreset_ex.restype = ctypes.c_int64
    lib.vo_attn_coreset_joint.argtypes = [_i32p, _i32p, ctypes.c_double, ctypes.c_int64, ctypes.c_int32, _f64p,
                                          _f64p, _f64p, _f64p, ctypes.c_int32, ctypes.c_double, ctypes.c_int64,
                                          _i64p, _f64p, _i32p, _i32p, ctypes.c_int]
    lib.vo_attn_coreset_joint.restype = ctypes.c_int64
    lib.vo_num_threads.argtypes = []
    lib.vo_num_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def _triple(x: Sequence[int]):
    a = (ctypes.c_int32 * 3)(*[int(e) for e in x])
    return a


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(ty)


def _rows(q_rows, default_n: int) -> Tuple[Optional[np.ndarray], int]:
    if q_rows is None:
        return None, default_n
    r = np.ascontiguousarray(np.asarray(q_rows, dtype=np.int64))
    return r, int(r.shape[0])


def num_threads() -> int:
    return int(_load().vo_num_threads())


def sta_token_mask(grid, tile, window) -> np.ndarray:
    """Algorithm 1's L x L mask by the literal double loop (tiny grids only)."""
    L = int(grid[0]) * int(grid[1]) * int(grid[2])
    M = np.zeros((L, L), dtype=np.uint8)
    _load().vo_sta_token_mask(_triple(grid), _triple(tile), _triple(window), _ptr(M, _u8p))
    return M


def sta_block_mask(grid, tile, window) -> np.ndarray:
    """Algorithm 1's test between tiles: uint8 [n_tiles, n_tiles]."""
    nt = [-(-int(g) // int(t)) for g, t in zip(grid, tile)]
    n = nt[0] * nt[1] * nt[2]
    BM = np.zeros((n, n), dtype=np.uint8)
    _load().vo_sta_block_mask(_triple(grid), _triple(tile), _triple(window), _ptr(BM, _u8p))
    return BM


def attn_full(Q, K, V, scale: float, q_rows=None, return_probs: bool = False):
    """Eq. 2 for one head: Q, K, V are [L, d]; returns O [nq, d] (and P [nq, L])."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    L, d = Q.shape
    rows, nq = _rows(q_rows, L)
    O = np.zeros((nq, d), dtype=np.float64)
    P = np.zeros((nq, L), dtype=np.float64) if return_probs else None
    rc = _load().vo_attn_full(L, d, _ptr(Q, _f64p), _ptr(K, _f64p), _ptr(V, _f64p), float(scale),
                              nq, _ptr(rows, _i64p), _ptr(O, _f64p), _ptr(P, _f64p))
    if rc != 0:
        raise MemoryError("vo_attn_full")
    return (O, P) if return_probs else O


def attn_sliding(grid, tile, window, Q, K, V, scale: float, q_rows=None,
                 return_probs: bool = False, text: int = 0):
    """Sliding tile attention (Algorithm 1's mask on Eq. 2) for one head.

    text: Q, K, V hold that many text tokens after the video tokens (joint sequence): text
    keys are visible to every query and text queries see every key."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    L, d = Q.shape
    assert L == int(grid[0]) * int(grid[1]) * int(grid[2]) + int(text)
    rows, nq = _rows(q_rows, L)
    O = np.zeros((nq, d), dtype=np.float64)
    P = np.zeros((nq, L), dtype=np.float64) if return_probs else None
    rc = _load().vo_attn_sliding_joint(_triple(grid), _triple(tile), _triple(window), int(text), d,
                                       _ptr(Q, _f64p), _ptr(K, _f64p), _ptr(V, _f64p), float(scale), nq,
                                       _ptr(rows, _i64p), _ptr(O, _f64p), _ptr(P, _f64p))
    if rc != 0:
        raise MemoryError("vo_attn_sliding")
    return (O, P) if return_probs else O


def coreset_len(grid, bucket, ratio: float) -> int:
    return int(_load().vo_coreset_len(_triple(grid), _triple(bucket), float(ratio)))


def coreset_select(grid, bucket, ratio: float, X, return_gap: bool = False):
    """Bucketed core-set selection on features X [L, dx].

    Returns (core_idx int32 [Lc], src_slot int32 [L]) and, if asked, the smallest
    gap between a pruned and a surviving score.
    """
    X = _f64(X)
    L, dx = X.shape
    assert L == int(grid[0]) * int(grid[1]) * int(grid[2])
    Lc = coreset_len(grid, bucket, ratio)
    core_idx = np.zeros(Lc, dtype=np.int32)
    src_slot = np.zeros(L, dtype=np.int32)
    gap = ctypes.c_double(0.0)
    got = _load().vo_coreset_select(_triple(grid), _triple(bucket), float(ratio), _ptr(X, _f64p),
                                    dx, _ptr(core_idx, _i32p), _ptr(src_slot, _i32p),
                                    ctypes.byref(gap))
    if got != Lc:
        raise RuntimeError(f"vo_coreset_select returned {got}, expected {Lc}")
    return (core_idx, src_slot, gap.value) if return_gap else (core_idx, src_slot)


def attn_coreset(grid, bucket, ratio: float, Q, K, V, scale: float, X=None, q_rows=None,
                 merge: bool = False, text: int = 0):
    """Core-set attention (unpool . attn . pool) for one head.

    X defaults to K.  merge: the centre's Q, K, V rows become the mean over the centre and
    the tokens pruned from its bucket.  text: Q, K, V (and X) hold that many text tokens after
    the video tokens; selection prunes video tokens only and every text token is kept.
    Returns (O [nq, d], core_idx [kept video tokens], src_slot [video tokens]).
    """
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    X = K if X is None else _f64(X)
    Ltot, d = Q.shape
    L = Ltot - int(text)
    assert L == int(grid[0]) * int(grid[1]) * int(grid[2]) and X.shape[0] >= L
    rows, nq = _rows(q_rows, Ltot)
    Lc = coreset_len(grid, bucket, ratio)
    O = np.zeros((nq, d), dtype=np.float64)
    core_idx = np.zeros(Lc, dtype=np.int32)
    src_slot = np.zeros(L, dtype=np.int32)
    got = _load().vo_attn_coreset_joint(_triple(grid), _triple(bucket), float(ratio), int(text), d,
                                        _ptr(Q, _f64p), _ptr(K, _f64p), _ptr(V, _f64p), _ptr(X, _f64p),
                                        X.shape[1], float(scale), nq, _ptr(rows, _i64p), _ptr(O, _f64p),
                                        _ptr(core_idx, _i32p), _ptr(src_slot, _i32p), int(bool(merge)))
    if got != Lc:
        raise RuntimeError(f"vo_attn_coreset returned {got}, expected {Lc}")
    return O, core_idx, src_slot


def router_gates(T, WR):
    """Router of Section 3.3: gates[h] = softmax(T @ WR[h]) (Eq. 3) and the branch Eq. 4 picks.

    T: [d_model]; WR: [heads, d_model, 3], gate order (full, sliding, core-set).  Returns
    (gates float64 [heads, 3], routes uint8 [heads]): sliding if its gate is strictly above
    both others, core-set likewise, full otherwise.
    """
    T = _f64(T)
    WR = _f64(WR)
    logits = np.einsum("c,hcr->hr", T, WR)
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    gates = e / e.sum(axis=1, keepdims=True)
    routes = np.zeros(gates.shape[0], dtype=np.uint8)
    a1, a2, a3 = gates[:, 0], gates[:, 1], gates[:, 2]
    routes[(a2 > a1) & (a2 > a3)] = 1
    routes[(a3 > a1) & (a3 > a2)] = 2
    return gates, routes


def soft_mixture(grid, tile, window, bucket, ratio, Q, K, V, scale, gates, q_rows=None, text: int = 0):
    """Eq. 5 for one head: gates[0] attn + gates[1] sliding-attn + gates[2] coreset-attn."""
    g = np.asarray(gates, dtype=np.float64)
    o_full = attn_full(Q, K, V, scale, q_rows=q_rows)
    o_sld = attn_sliding(grid, tile, window, Q, K, V, scale, q_rows=q_rows, text=text)
    o_core, _, _ = attn_coreset(grid, bucket, ratio, Q, K, V, scale, q_rows=q_rows, text=text)
    return g[0] * o_full + g[1] * o_sld + g[2] * o_core
