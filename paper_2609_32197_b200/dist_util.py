"""Multi-process plumbing for the benchmark: the path shards by independent replicas (one workload per
GPU, no data-path collective), so all that crosses ranks is the timing reduction."""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import synth


def replica_workload(wl: synth.Workload, rank: int) -> synth.Workload:
    """The workload rank `rank` runs: same shapes, its own seed (rank 0 keeps the named workload)."""
    if rank == 0:
        return wl
    return synth.Workload(wl.name, wl.heads, wl.head_dim, wl.grid, wl.n_text, wl.block, wl.topk_abs,
                          wl.topk_pct, wl.ranks, wl.placements, seed=wl.seed + rank)


def head_shard(heads: int, rank: int, world: int):
    """Heads [begin, end) of ONE layer that rank `rank` of `world` takes (strong scaling by heads: every step of
    the path is independent per head, so the shards need no exchange and their outputs concatenate)."""
    return (rank * heads) // world, ((rank + 1) * heads) // world


def reduce_over_ranks(times_ms: dict, totals: dict, device="cpu"):
    """Device-timed milliseconds -> MAX over ranks; work totals (flops, launches) -> SUM over ranks.
    With a single process (no process group) the inputs come back unchanged."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return dict(times_ms), dict(totals)
    tk, sk = sorted(times_ms), sorted(totals)
    t = torch.tensor([float(times_ms[k]) for k in tk], dtype=torch.float64, device=device)
    s = torch.tensor([float(totals[k]) for k in sk], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return dict(zip(tk, t.tolist())), dict(zip(sk, s.tolist()))
