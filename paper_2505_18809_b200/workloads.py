"""Seeded synthetic workloads: shapes, routes and Q/K/V values.

This module holds no attention arithmetic; it only makes inputs.  Both the CUDA
library's callers and the CPU checker are fed from the SAME buffers made here.

Shapes follow the latent grids of the video DiTs the paper measures
(Wan 2.1 1.3B at 480p, HunyuanVideo at 720p, Wan 2.1 14B at 720p); values are a
spatially smooth Gaussian field plus noise, so that neighbouring tokens are
similar, which is what bucketed core-set selection relies on (Section 1,
"high intra-sequence redundancy").
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import torch

ROUTE_FULL, ROUTE_SLIDING, ROUTE_CORESET = 0, 1, 2


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    grid: Tuple[int, int, int]          # latent (T, H, W)
    heads: int
    d: int
    tile: Tuple[int, int, int]
    window: Tuple[int, int, int]        # in tiles
    ratio: float
    routes: Tuple[int, ...]
    seed: int
    smooth: bool                        # False: plain N(0,1)
    B: int = 1
    bucket: Tuple[int, int, int] = (2, 3, 2)
    merge: bool = False                 # core-set heads merge pruned tokens into the centre (mean)
    text: int = 0                       # text tokens after the video tokens of every head (MMDiT joint sequence)

    @property
    def L(self) -> int:
        """Video tokens per head."""
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def rows(self) -> int:
        """Rows per head of Q, K, V, O: video tokens, then text tokens."""
        return self.L + self.text


def apportion_routes(heads: int, fractions: Sequence[float], seed: int) -> Tuple[int, ...]:
    """Largest-remainder split of `heads` into (full, sliding, coreset) counts,
    then a seeded shuffle of the head positions."""
    raw = [f * heads for f in fractions]
    cnt = [int(math.floor(x)) for x in raw]
    rem = sorted(range(3), key=lambda i: (-(raw[i] - cnt[i]), i))
    for i in rem[: heads - sum(cnt)]:
        cnt[i] += 1
    routes = [ROUTE_FULL] * cnt[0] + [ROUTE_SLIDING] * cnt[1] + [ROUTE_CORESET] * cnt[2]
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(heads, generator=g).tolist()
    return tuple(routes[p] for p in perm)


def config(name: str) -> Workload:
    """The named benchmark configurations."""
    if name == "tiny":
        return Workload("tiny", (4, 8, 8), 2, 64, (2, 4, 4), (3, 3, 3), 0.25,
                        (ROUTE_SLIDING, ROUTE_CORESET), 0, False)
    if name == "wan1.3b-480p":
        return Workload(name, (21, 30, 52), 12, 128, (4, 4, 4), (3, 3, 3), 0.5,
                        apportion_routes(12, (1 / 3, 1 / 3, 1 / 3), 1), 1, True)
    if name == "hunyuan-720p":
        return Workload(name, (33, 45, 80), 24, 128, (4, 8, 8), (3, 3, 3), 0.5,
                        apportion_routes(24, (0.2, 0.5, 0.3), 2), 2, True)
    if name == "wan14b-720p":
        return Workload(name, (21, 45, 80), 40, 128, (4, 8, 8), (3, 3, 3), 0.25,
                        apportion_routes(40, (0.0, 0.8, 0.2), 3), 3, True)
    if name == "hunyuan-720p-text256":
        # second workload: the MMDiT joint sequence of HunyuanVideo, 256 text tokens after the video tokens
        return Workload(name, (33, 45, 80), 24, 128, (4, 8, 8), (3, 3, 3), 0.5,
                        apportion_routes(24, (0.2, 0.5, 0.3), 2), 2, True, 1, (2, 3, 2), False, 256)
    if name == "hunyuan-30x45x80-tile6x9x8":
        # the window the paper prints for HunyuanVideo (18 x 27 x 24 = 3 tiles of 6 x 9 x 8 on the
        # 30 x 45 x 80 latent, Appendix A.2): 432-token tiles, cut into four boxes of 108
        return Workload(name, (30, 45, 80), 24, 128, (6, 9, 8), (3, 3, 3), 0.5,
                        apportion_routes(24, (0.2, 0.5, 0.3), 2), 2, True)
    if name == "hunyuan-720p-3h":
        # profiling case: the HunyuanVideo-720p grid with one head per route, so that a
        # counter capture of one launch stays short while the inputs still exceed L2
        return Workload(name, (33, 45, 80), 3, 128, (4, 8, 8), (3, 3, 3), 0.5,
                        (ROUTE_FULL, ROUTE_SLIDING, ROUTE_CORESET), 2, True)
    if name == "hunyuan-720p-8c":
        # profiling case for the memory-bound stages: eight core-set heads, nothing else
        return Workload(name, (33, 45, 80), 8, 128, (4, 8, 8), (3, 3, 3), 0.5,
                        (ROUTE_CORESET,) * 8, 2, True)
    raise KeyError(name)


CONFIG_NAMES = ("tiny", "wan1.3b-480p", "hunyuan-720p", "wan14b-720p")
JOINT_NAMES = ("hunyuan-720p-text256", "hunyuan-30x45x80-tile6x9x8")  # further workloads bench.py accepts
PROFILE_NAMES = ("hunyuan-720p-3h", "hunyuan-720p-8c")


def route_mix_sweep() -> List[Workload]:
    """HunyuanVideo-720p shape; fraction of full heads 0/.25/.5/1, the rest split
    evenly between sliding and core-set; core-set ratio .25/.5; seeds 4..11."""
    out = []
    for fi, f in enumerate((0.0, 0.25, 0.5, 1.0)):
        for ri, r in enumerate((0.25, 0.5)):
            seed = 4 + 2 * fi + ri
            routes = apportion_routes(24, (f, (1 - f) / 2, (1 - f) / 2), seed)
            out.append(Workload(f"hunyuan-720p-full{f:g}-r{r:g}", (33, 45, 80), 24, 128, (4, 8, 8),
                                (3, 3, 3), r, routes, seed, True))
    return out


def _smooth_field(n_chan: int, grid, g: torch.Generator, device) -> torch.Tensor:
    """[n_chan, T, H, W]: N(0,1) blurred by a 5x5x5 box mean (cut at the borders,
    divided by the number of cells really covered), times sqrt(125), plus 0.3*N(0,1)."""
    T, H, W = grid
    x = torch.randn((n_chan, 1, T, H, W), generator=g, device=device, dtype=torch.float32)
    ones = torch.ones((1, 1, 5, 5, 5), device=device, dtype=torch.float32)
    cells = torch.nn.functional.conv3d(torch.ones((1, 1, T, H, W), device=device), ones, padding=2)
    blur = torch.nn.functional.conv3d(x, ones, padding=2) / cells
    blur = blur * math.sqrt(125.0)
    blur += 0.3 * torch.randn((n_chan, 1, T, H, W), generator=g, device=device,
                              dtype=torch.float32)
    return blur[:, 0]


def make_qkv(wl: Workload, device="cpu", heads: Optional[Sequence[int]] = None):
    """Q, K, V as bf16 [B, heads, L + text, d] on `device`, video token order i = (t*H + h)*W + w,
    text tokens (plain N(0,1)) after them.

    One generator per (tensor, batch, head), seeded from the workload seed, so a
    subset of heads can be made without the rest (`heads`: which heads to fill; the
    others stay zero).  CPU and CUDA generators give different streams: make the
    tensors once and hand the same buffers to every consumer.
    """
    dev = torch.device(device)
    T, H, W = wl.grid
    L = wl.L
    out = []
    for ti in range(3):
        x = torch.zeros((wl.B, wl.heads, L + wl.text, wl.d), dtype=torch.bfloat16, device=dev)
        for b in range(wl.B):
            for h in (range(wl.heads) if heads is None else heads):
                g = torch.Generator(device=dev)
                g.manual_seed(((wl.seed * 3 + ti) * 64 + b) * 4096 + h)
                if wl.smooth:
                    f = _smooth_field(wl.d, wl.grid, g, dev)            # [d, T, H, W]
                    f = f.reshape(wl.d, L).t()
                else:
                    f = torch.randn((L, wl.d), generator=g, device=dev, dtype=torch.float32)
                x[b, h, :L] = f.to(torch.bfloat16)
                if wl.text:
                    x[b, h, L:] = torch.randn((wl.text, wl.d), generator=g, device=dev,
                                              dtype=torch.float32).to(torch.bfloat16)
        out.append(x)
    return tuple(out)
