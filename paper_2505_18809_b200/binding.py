"""Thin ctypes binding of libvorta.so: argument marshalling only.

The module-level functions carry the names of the C entry points (see
include/vorta.h) and take raw integers for device pointers; `Plan` wraps them for
torch tensors.  Nothing here computes: every step runs in the library's kernels.
The library must be present; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvorta.so")

VORTA_OK = 0
VORTA_ERR_INVALID_ARG, VORTA_ERR_UNSUPPORTED, VORTA_ERR_ALIGNMENT = 1, 2, 3
VORTA_ERR_WORKSPACE, VORTA_ERR_CUDA, VORTA_ERR_TIMEOUT, VORTA_ERR_INTERNAL = 4, 5, 6, 7
VORTA_ROUTE_FULL, VORTA_ROUTE_SLIDING, VORTA_ROUTE_CORESET = 0, 1, 2
VORTA_PLAN_HOST_ONLY = 1
VORTA_PLAN_POOL_MERGE = 2
VORTA_KERNEL_TCGEN05, VORTA_KERNEL_SIMT, VORTA_KERNEL_PAIR, VORTA_KERNEL_AUTO = 0, 1, 2, 3

EXPORTS = (
    "vorta_plan_create", "vorta_plan_set_routes", "vorta_plan_destroy", "vorta_plan_info",
    "vorta_plan_block_mask", "vorta_plan_set_kernel", "vorta_coreset_select",
    "vorta_routed_attention", "vorta_routed_attention_host", "vorta_plan_set_profiling",
    "vorta_plan_stage_ms", "vorta_plan_stage_ms_at", "vorta_plan_last_launches", "vorta_device_status",
    "vorta_status_string", "vorta_routed_attention_static", "vorta_plan_device",
    "vorta_router_gates", "vorta_soft_mixture", "vorta_shard_heads", "vorta_plan_kernel_in_use",
    "vorta_plan_attention_ms_at",
)
VORTA_STATIC_WORKSPACE_BYTES = 16 * 1024 * 1024


class vorta_plan_desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("heads", ctypes.c_int32), ("T", ctypes.c_int32),
                ("H", ctypes.c_int32), ("W", ctypes.c_int32), ("d", ctypes.c_int32),
                ("tile", ctypes.c_int32 * 3), ("window", ctypes.c_int32 * 3),
                ("bucket", ctypes.c_int32 * 3), ("coreset_ratio", ctypes.c_float),
                ("softmax_scale", ctypes.c_float), ("routes", ctypes.POINTER(ctypes.c_uint8)),
                ("flags", ctypes.c_int32), ("device", ctypes.c_int32), ("text_tokens", ctypes.c_int32)]


class vorta_plan_info_t(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int64), ("Lc", ctypes.c_int64),
                ("tiles_per_axis", ctypes.c_int32 * 3), ("n_tiles", ctypes.c_int32),
                ("n_buckets", ctypes.c_int32), ("kv_tiles_per_q_tile", ctypes.c_int32),
                ("n_full", ctypes.c_int32), ("n_sliding", ctypes.c_int32),
                ("n_coreset", ctypes.c_int32), ("workspace_bytes", ctypes.c_int64),
                ("workspace_bytes_max", ctypes.c_int64),
                ("host_call_scratch_bytes", ctypes.c_int64),
                ("mixture_workspace_bytes", ctypes.c_int64),
                ("flops_full_head", ctypes.c_double), ("flops_sliding_head", ctypes.c_double),
                ("flops_coreset_head", ctypes.c_double), ("flops_layer", ctypes.c_double),
                ("flops_issued_layer", ctypes.c_double), ("n_work_items", ctypes.c_int64),
                ("select_bytes_head", ctypes.c_int64), ("gather_bytes_head", ctypes.c_int64),
                ("scatter_bytes_head", ctypes.c_int64), ("text_tokens", ctypes.c_int64)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load libvorta.so (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2505_18809_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    L.vorta_plan_create.argtypes = [ctypes.POINTER(vorta_plan_desc), ctypes.POINTER(vp)]
    L.vorta_plan_set_routes.argtypes = [vp, ctypes.POINTER(ctypes.c_uint8), i32]
    L.vorta_plan_destroy.argtypes = [vp]
    L.vorta_plan_info.argtypes = [vp, ctypes.POINTER(vorta_plan_info_t)]
    L.vorta_plan_block_mask.argtypes = [vp, vp]
    L.vorta_plan_set_kernel.argtypes = [vp, i32]
    L.vorta_plan_kernel_in_use.argtypes = [vp]
    L.vorta_plan_kernel_in_use.restype = i32
    L.vorta_coreset_select.argtypes = [vp, vp, i32, i32, vp, vp, vp]
    L.vorta_routed_attention.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, ctypes.c_size_t, vp]
    L.vorta_routed_attention_host.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.vorta_routed_attention_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp]
    L.vorta_plan_device.argtypes = [vp, ctypes.POINTER(i32)]
    L.vorta_router_gates.argtypes = [vp, vp, i32, i32, vp, vp, vp]
    L.vorta_soft_mixture.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.vorta_plan_set_profiling.argtypes = [vp, i32]
    L.vorta_plan_stage_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float * 4)]
    L.vorta_plan_stage_ms_at.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_float * 4)]
    L.vorta_plan_attention_ms_at.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_float * 2)]
    L.vorta_plan_last_launches.argtypes = [vp, ctypes.POINTER(i32)]
    L.vorta_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    L.vorta_status_string.argtypes = [ctypes.c_int]
    L.vorta_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "vorta_status_string":
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


class VortaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {vorta_status_string(status)} (status {status})")


def _check(status: int, where: str) -> None:
    if status != VORTA_OK:
        raise VortaError(status, where)


# ------------------------------------------------------------------ C-named functions
def vorta_status_string(status: int) -> str:
    return lib().vorta_status_string(int(status)).decode()


def vorta_plan_create(desc: vorta_plan_desc) -> int:
    """Returns the plan handle (an integer address); raises VortaError on failure."""
    out = ctypes.c_void_p()
    _check(lib().vorta_plan_create(ctypes.byref(desc), ctypes.byref(out)), "vorta_plan_create")
    return out.value


def vorta_plan_set_routes(plan: int, routes: Sequence[int]) -> None:
    arr = (ctypes.c_uint8 * len(routes))(*[int(r) for r in routes])
    _check(lib().vorta_plan_set_routes(plan, arr, len(routes)), "vorta_plan_set_routes")


def vorta_plan_destroy(plan: int) -> None:
    _check(lib().vorta_plan_destroy(plan), "vorta_plan_destroy")


def vorta_plan_info(plan: int) -> vorta_plan_info_t:
    info = vorta_plan_info_t()
    _check(lib().vorta_plan_info(plan, ctypes.byref(info)), "vorta_plan_info")
    return info


def vorta_shard_heads(plan: int, heads: int, n_ranks: int):
    """(rank_of_head int32 [heads], rank_flops float64 [n_ranks]) of the current routes."""
    rank_of_head = np.zeros(heads, dtype=np.int32)
    rank_flops = np.zeros(n_ranks, dtype=np.float64)
    _check(lib().vorta_shard_heads(plan, int(n_ranks), rank_of_head.ctypes.data_as(ctypes.c_void_p),
                                   rank_flops.ctypes.data_as(ctypes.c_void_p)), "vorta_shard_heads")
    return rank_of_head, rank_flops


def vorta_plan_block_mask(plan: int, n_tiles: int) -> np.ndarray:
    out = np.zeros((n_tiles, n_tiles), dtype=np.uint8)
    _check(lib().vorta_plan_block_mask(plan, out.ctypes.data), "vorta_plan_block_mask")
    return out


def vorta_plan_set_kernel(plan: int, kernel: int) -> None:
    _check(lib().vorta_plan_set_kernel(plan, kernel), "vorta_plan_set_kernel")


def vorta_plan_kernel_in_use(plan: int) -> int:
    return int(lib().vorta_plan_kernel_in_use(plan))


def vorta_coreset_select(plan: int, X_ptr: int, Hx: int, dx: int, core_idx_ptr: int,
                         src_slot_ptr: int, stream: int = 0) -> None:
    _check(lib().vorta_coreset_select(plan, X_ptr, Hx, dx, core_idx_ptr, src_slot_ptr, stream),
           "vorta_coreset_select")


def vorta_routed_attention(plan: int, Q_ptr: int, K_ptr: int, V_ptr: int, O_ptr: int,
                           X_ptr: Optional[int], Hx: int, workspace_ptr: Optional[int],
                           workspace_bytes: int, stream: int = 0) -> None:
    _check(lib().vorta_routed_attention(plan, Q_ptr, K_ptr, V_ptr, O_ptr, X_ptr, Hx,
                                        workspace_ptr, workspace_bytes, stream),
           "vorta_routed_attention")


def vorta_routed_attention_host(plan: int, Q_ptr: int, K_ptr: int, V_ptr: int, O_ptr: int,
                                scratch_ptr: int, scratch_bytes: int, stream: int = 0) -> None:
    _check(lib().vorta_routed_attention_host(plan, Q_ptr, K_ptr, V_ptr, O_ptr, scratch_ptr,
                                             scratch_bytes, stream),
           "vorta_routed_attention_host")


def vorta_routed_attention_static(plan: int, Q_ptr: int, K_ptr: int, V_ptr: int, O_ptr: int,
                                  X_ptr: Optional[int] = None, Hx: int = 0, stream: int = 0) -> None:
    """The layer with the library's built-in scratch array: for callers that may not allocate."""
    _check(lib().vorta_routed_attention_static(plan, Q_ptr, K_ptr, V_ptr, O_ptr, X_ptr, Hx, stream),
           "vorta_routed_attention_static")


def vorta_plan_device(plan: int) -> int:
    d = ctypes.c_int32()
    _check(lib().vorta_plan_device(plan, ctypes.byref(d)), "vorta_plan_device")
    return d.value


def vorta_router_gates(T_ptr: int, WR_ptr: int, d_model: int, heads: int, gates_ptr: int, routes_ptr: int,
                       stream: int = 0) -> None:
    _check(lib().vorta_router_gates(T_ptr, WR_ptr, d_model, heads, gates_ptr, routes_ptr, stream),
           "vorta_router_gates")


def vorta_soft_mixture(plan: int, Q_ptr: int, K_ptr: int, V_ptr: int, gates_ptr: int, O_ptr: int,
                       workspace_ptr: int, workspace_bytes: int, stream: int = 0) -> None:
    _check(lib().vorta_soft_mixture(plan, Q_ptr, K_ptr, V_ptr, gates_ptr, O_ptr, workspace_ptr,
                                    workspace_bytes, stream), "vorta_soft_mixture")


def vorta_plan_set_profiling(plan: int, on: bool) -> None:
    _check(lib().vorta_plan_set_profiling(plan, int(bool(on))), "vorta_plan_set_profiling")


def vorta_plan_stage_ms(plan: int):
    ms = (ctypes.c_float * 4)()
    _check(lib().vorta_plan_stage_ms(plan, ctypes.byref(ms)), "vorta_plan_stage_ms")
    return [float(x) for x in ms]


def vorta_plan_stage_ms_at(plan: int, calls_back: int):
    ms = (ctypes.c_float * 4)()
    _check(lib().vorta_plan_stage_ms_at(plan, calls_back, ctypes.byref(ms)), "vorta_plan_stage_ms_at")
    return [float(x) for x in ms]


def vorta_plan_attention_ms_at(plan: int, calls_back: int):
    ms = (ctypes.c_float * 2)()
    _check(lib().vorta_plan_attention_ms_at(plan, calls_back, ctypes.byref(ms)), "vorta_plan_attention_ms_at")
    return [float(x) for x in ms]


def vorta_plan_last_launches(plan: int) -> int:
    n = ctypes.c_int32()
    _check(lib().vorta_plan_last_launches(plan, ctypes.byref(n)), "vorta_plan_last_launches")
    return n.value


def vorta_device_status(plan: int, stream: int = 0) -> int:
    """Synchronises the stream; returns 0, or raises VortaError(TIMEOUT) carrying the code."""
    code = ctypes.c_int32()
    st = lib().vorta_device_status(plan, stream, ctypes.byref(code))
    if st == VORTA_ERR_TIMEOUT:
        raise VortaError(st, f"vorta_device_status (device code {code.value})")
    _check(st, "vorta_device_status")
    return code.value


def make_desc(B, heads, grid, d, tile, window, ratio, routes, bucket=(0, 0, 0), scale=0.0,
              flags=0, device=-1, text=0):
    """Fill a vorta_plan_desc; keeps the routes array alive on the returned object."""
    desc = vorta_plan_desc()
    desc.B, desc.heads = int(B), int(heads)
    desc.T, desc.H, desc.W = (int(x) for x in grid)
    desc.d = int(d)
    desc.tile = (ctypes.c_int32 * 3)(*[int(x) for x in tile])
    desc.window = (ctypes.c_int32 * 3)(*[int(x) for x in window])
    desc.bucket = (ctypes.c_int32 * 3)(*[int(x) for x in bucket])
    desc.coreset_ratio = float(ratio)
    desc.softmax_scale = float(scale)
    arr = (ctypes.c_uint8 * len(routes))(*[int(r) for r in routes])
    desc._routes_keepalive = arr
    desc.routes = ctypes.cast(arr, ctypes.POINTER(ctypes.c_uint8))
    desc.flags, desc.device = int(flags), int(device)
    desc.text_tokens = int(text)
    return desc


# ------------------------------------------------------------------ torch convenience
class Plan:
    """Owns one vorta_plan; methods take torch CUDA tensors and pass their pointers on."""

    def __init__(self, B, heads, grid, d, tile, window, ratio, routes, bucket=(0, 0, 0),
                 scale=0.0, host_only=False, device=-1, merge=False, text=0):
        flags = (VORTA_PLAN_HOST_ONLY if host_only else 0) | (VORTA_PLAN_POOL_MERGE if merge else 0)
        self.desc = make_desc(B, heads, grid, d, tile, window, ratio, routes, bucket, scale, flags, device, text)
        self.handle = vorta_plan_create(self.desc)
        self.B, self.heads, self.grid, self.d = B, heads, tuple(grid), d
        self._workspace = None

    @classmethod
    def from_workload(cls, wl, host_only=False, device=-1):
        return cls(wl.B, wl.heads, wl.grid, wl.d, wl.tile, wl.window, wl.ratio, wl.routes,
                   wl.bucket, 0.0, host_only, device, getattr(wl, "merge", False), getattr(wl, "text", 0))

    def close(self):
        if getattr(self, "handle", None):
            vorta_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def info(self) -> vorta_plan_info_t:
        return vorta_plan_info(self.handle)

    def set_routes(self, routes):
        vorta_plan_set_routes(self.handle, list(routes))

    def set_kernel(self, kernel: int):
        vorta_plan_set_kernel(self.handle, kernel)

    def kernel_in_use(self) -> int:
        """The VORTA_KERNEL_* the routed call runs with the current routes (AUTO resolved)."""
        return vorta_plan_kernel_in_use(self.handle)

    def set_profiling(self, on: bool):
        vorta_plan_set_profiling(self.handle, on)

    def stage_ms(self, calls_back: int = 0):
        """[select, gather, attention, scatter] milliseconds of a profiled call."""
        return vorta_plan_stage_ms_at(self.handle, calls_back)

    def attention_ms(self, calls_back: int = 0):
        """[first attention kernel, single-CTA kernel after the pair kernel (0 if one launch)] milliseconds."""
        return vorta_plan_attention_ms_at(self.handle, calls_back)

    def last_launches(self) -> int:
        return vorta_plan_last_launches(self.handle)

    def block_mask(self) -> np.ndarray:
        return vorta_plan_block_mask(self.handle, self.info.n_tiles)

    def device_status(self, stream: int = 0) -> int:
        return vorta_device_status(self.handle, stream)

    @staticmethod
    def _stream() -> int:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)

    def coreset_select(self, X):
        """X: bf16 CUDA [B, Hx, L + text, dx] -> (core_idx int32 [B, Hx, Lc], src_slot int32 [B, Hx, L]);
        only the L video rows of X are looked at."""
        import torch
        assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous()
        B, Hx, rows, dx = X.shape
        info = self.info
        assert B == self.B and rows == info.L + info.text_tokens
        core_idx = torch.empty((B, Hx, info.Lc), dtype=torch.int32, device=X.device)
        src_slot = torch.empty((B, Hx, info.L), dtype=torch.int32, device=X.device)
        vorta_coreset_select(self.handle, X.data_ptr(), Hx, dx, core_idx.data_ptr(),
                             src_slot.data_ptr(), self._stream())
        return core_idx, src_slot

    def workspace(self, device):
        """A cached device workspace large enough for the current routes."""
        import torch
        need = int(self.info.workspace_bytes)
        if need == 0:
            return None
        if self._workspace is None or self._workspace.numel() < need:
            self._workspace = torch.empty(need, dtype=torch.uint8, device=device)
        return self._workspace

    def routed_attention(self, Q, K, V, O=None, X=None, workspace=None):
        """Q, K, V: bf16 CUDA [B, heads, L + text, d] -> O (same shape)."""
        import torch
        info = self.info
        for t in (Q, K, V):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
            assert tuple(t.shape) == (self.B, self.heads, info.L + info.text_tokens, self.d)
        if O is None:
            O = torch.empty_like(Q)
        ws = workspace if workspace is not None else self.workspace(Q.device)
        Hx = 0 if X is None else X.shape[1]
        vorta_routed_attention(self.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(),
                               None if X is None else X.data_ptr(), Hx,
                               None if ws is None else ws.data_ptr(),
                               0 if ws is None else ws.numel(), self._stream())
        return O

    def soft_mixture(self, Q, K, V, gates, O=None, workspace=None):
        """gates: f32 CUDA [heads, 3]; every head runs all three branches (Eq. 5)."""
        import torch
        if O is None:
            O = torch.empty_like(Q)
        need = int(self.info.mixture_workspace_bytes)
        ws = workspace if workspace is not None else torch.empty(need, dtype=torch.uint8, device=Q.device)
        vorta_soft_mixture(self.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(), gates.data_ptr(),
                           O.data_ptr(), ws.data_ptr(), ws.numel(), self._stream())
        return O

    def routed_attention_host(self, Qh, Kh, Vh, Oh, scratch):
        """Host (pinned) tensors in and out; `scratch` is a uint8 CUDA tensor."""
        vorta_routed_attention_host(self.handle, Qh.data_ptr(), Kh.data_ptr(), Vh.data_ptr(),
                                    Oh.data_ptr(), scratch.data_ptr(), scratch.numel(),
                                    self._stream())
        return Oh


def router_gates(T, WR):
    """T: f32 CUDA [d_model]; WR: f32 CUDA [heads, d_model, 3] -> (gates f32 [heads, 3], routes uint8 [heads])."""
    import torch
    heads, d_model, three = WR.shape
    assert three == 3 and T.shape == (d_model,) and T.is_cuda and WR.is_contiguous()
    gates = torch.empty((heads, 3), dtype=torch.float32, device=T.device)
    routes = torch.empty((heads,), dtype=torch.uint8, device=T.device)
    vorta_router_gates(T.data_ptr(), WR.data_ptr(), d_model, heads, gates.data_ptr(), routes.data_ptr(),
                       int(torch.cuda.current_stream().cuda_stream))
    return gates, routes
