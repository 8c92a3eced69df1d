"""Seeded synthetic inputs shaped like video-DiT attention layers.

This module is the only code shared by the CPU oracle's tests and the CUDA path's tests/bench.  It
holds none of the method's arithmetic: it only draws Q/K/V and a shuffled block order.  Everything
is generated with torch ops, so the same recipe runs on the CPU (parity tests: generate once, hand
the same bits to both sides) or directly on the GPU (benchmarks).

Recipe (per head h):
  * a video token at grid position (t, y, x) gets a 48-feature vector: sin and cos of
    2*pi * 2^m * coord / extent for the three coordinates and m = 0..7;
  * a text token gets a 48-feature vector drawn N(0, 1/2) (same energy per feature);
  * W_h is a random d x 48 matrix, entries N(0, 1/48), shared by Q and K of that head, so that
    q.k peaks for tokens that are close in every coordinate (diagonal and multi-diagonal block
    structure);
  * Q = 2 W_h f + N(0, 0.5^2), K = 2 W_h f + N(0, 0.5^2) (independent noise), V ~ N(0, 1);
  * all rounded to bf16.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

N_FREQ = 8
N_FEAT = 3 * 2 * N_FREQ


@dataclass(frozen=True)
class Workload:
    name: str
    heads: int
    head_dim: int
    grid: tuple  # (T, Hg, Wg)
    n_text: int
    block: int
    topk_abs: int | None  # kept video blocks per row, absolute ...
    topk_pct: tuple | None  # ... or percentages of the video blocks (first entry = default)
    ranks: int
    placements: tuple = ("contiguous",)
    seed: int = 0

    @property
    def n_video(self) -> int:
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def n_tokens(self) -> int:
        return self.n_video + self.n_text

    @property
    def n_blocks(self) -> int:
        return (self.n_tokens + self.block - 1) // self.block

    @property
    def frame_tokens(self) -> int:
        return self.grid[1] * self.grid[2]

    @property
    def nb_video(self) -> int:
        """Blocks that hold no text token."""
        if self.n_text == 0:
            return self.n_blocks
        return self.n_video // self.block


WORKLOADS = {
    "tiny": Workload("tiny", 2, 64, (4, 32, 32), 0, 64, 16, None, 4),
    "mid": Workload("mid", 24, 128, (8, 48, 64), 0, 64, None, (15,), 4),
    "cog": Workload("cog", 48, 64, (13, 30, 45), 226, 64, None, (20,), 8, ("shuffle",)),
    "wan": Workload("wan", 40, 128, (21, 45, 80), 0, 128, None, (10,), 8, ("contiguous", "periodic")),
    "hunyuan": Workload("hunyuan", 24, 128, (33, 45, 80), 0, 128, None, (10, 5, 25), 8),
}


def features(wl: Workload, device="cpu") -> torch.Tensor:
    """[N][48] fp32 feature rows (video tokens in row-major (t, y, x) order, then text tokens)."""
    T, Hg, Wg = wl.grid
    t = torch.arange(T, device=device, dtype=torch.float64).view(T, 1, 1).expand(T, Hg, Wg)
    y = torch.arange(Hg, device=device, dtype=torch.float64).view(1, Hg, 1).expand(T, Hg, Wg)
    x = torch.arange(Wg, device=device, dtype=torch.float64).view(1, 1, Wg).expand(T, Hg, Wg)
    cols = []
    for coord, extent in ((t, T), (y, Hg), (x, Wg)):
        c = coord.reshape(-1)
        for m in range(N_FREQ):
            ang = 2.0 * math.pi * (2.0 ** m) * c / float(extent)
            cols.append(torch.sin(ang))
            cols.append(torch.cos(ang))
    f = torch.stack(cols, dim=1).to(torch.float32)
    if wl.n_text > 0:
        g = torch.Generator(device="cpu").manual_seed(wl.seed * 7919 + 17)
        ft = torch.randn(wl.n_text, N_FEAT, generator=g, dtype=torch.float32) * math.sqrt(0.5)
        f = torch.cat([f, ft.to(device)], dim=0)
    return f


def make_qkv(wl: Workload, device="cpu", heads: int | None = None, head_begin: int = 0):
    """-> Q, K, V bf16 tensors of shape [H][N][d] on ``device`` (H = wl.heads unless overridden); output head
    h holds the workload's head ``head_begin + h`` (a shard of the heads draws the same values as the whole).

    Random draws are made by a CPU generator per (seed, head, tensor) when device is the CPU and by
    the device's generator otherwise; values for a given device type are reproducible."""
    H = wl.heads if heads is None else heads
    N, d = wl.n_tokens, wl.head_dim
    f = features(wl, device)
    Q = torch.empty(H, N, d, dtype=torch.bfloat16, device=device)
    K = torch.empty_like(Q)
    V = torch.empty_like(Q)
    dev = torch.device(device)
    for h in range(H):
        g = torch.Generator(device=dev.type if dev.type == "cpu" else dev)
        g.manual_seed(wl.seed * 1000003 + (head_begin + h) * 101 + 1)
        W = torch.randn(d, N_FEAT, generator=g, dtype=torch.float32, device=device) / math.sqrt(N_FEAT)
        base = 2.0 * (f @ W.t())
        Q[h] = (base + 0.5 * torch.randn(N, d, generator=g, dtype=torch.float32, device=device)).to(torch.bfloat16)
        K[h] = (base + 0.5 * torch.randn(N, d, generator=g, dtype=torch.float32, device=device)).to(torch.bfloat16)
        V[h] = torch.randn(N, d, generator=g, dtype=torch.float32, device=device).to(torch.bfloat16)
    return Q, K, V


def shuffled_placement(n_blocks: int, ranks: int, seed: int = 1) -> torch.Tensor:
    """Seeded random placement: a random permutation of the blocks is cut into ``ranks`` contiguous
    runs; the block at shuffled position q goes to rank floor(q*ranks/n_blocks).  int32 [NB], CPU."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    perm = torch.randperm(n_blocks, generator=g)
    out = torch.empty(n_blocks, dtype=torch.int32)
    pos = torch.arange(n_blocks, dtype=torch.int64)
    out[perm] = ((pos * ranks) // n_blocks).to(torch.int32)
    return out
