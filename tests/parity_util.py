"""Shared helpers of the GPU parity tests: run the three C-ABI calls on one set of inputs and compare
every output with the CPU oracle (bit-exact for integers and bytes, tolerance for attention)."""
from __future__ import annotations

import numpy as np
import torch

ATTN_MAX_ABS = 2e-2   # tolerance on |O_gpu - O_oracle|, bf16 inputs, fp32/fp64 oracle
ATTN_MEAN_ABS = 2e-3


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy().view(np.uint32)


def to_layout(x_hnd: torch.Tensor, layout: str) -> torch.Tensor:
    """[H][N][d] -> device tensor in the requested memory layout (returned in its storage order)."""
    if layout == "HND":
        return x_hnd.contiguous()
    return x_hnd.permute(1, 0, 2).contiguous()  # [N][H][d]


def from_layout(x: torch.Tensor, layout: str) -> torch.Tensor:
    return x if layout == "HND" else x.permute(1, 0, 2)


def gpu_block_mask(binding, shape, Qd, Kd, k, ws, with_pooled=True):
    outs = binding.alloc_mask_outputs(shape, k, with_list=True, with_pooled=with_pooled)
    binding.sparsp_block_mask(shape, Qd, Kd, k, outs["mask"], outs["kv_list"], outs["kv_count"],
                              outs["pooled_q"], outs["pooled_k"], ws)
    torch.cuda.synchronize()
    return outs


def check_mask(oracle, binding, shape, Q, K, Qd, Kd, k, n_text, ws):
    """Q, K: CPU [H][N][d] bf16 (oracle side); Qd, Kd: the same bits on the device."""
    b = shape.block
    ref = oracle.block_mask(Q, K, b, k, n_text)
    got = gpu_block_mask(binding, shape, Qd, Kd, k, ws)
    assert np.array_equal(got["pooled_q"][0].cpu().numpy().view(np.uint32), ref["pq"].view(np.uint32)), "pooled Q"
    assert np.array_equal(got["pooled_k"][0].cpu().numpy().view(np.uint32), ref["pk"].view(np.uint32)), "pooled K"
    gm = u32(got["mask"][0])
    if not np.array_equal(gm, ref["mask"]):
        bad = np.argwhere((gm != ref["mask"]).any(axis=2))
        # near-tie audit: would an fp64 score order explain the difference?
        raise AssertionError(f"mask differs on {len(bad)} rows, first (h, i) = {bad[0].tolist()}")
    assert np.array_equal(got["kv_list"][0].cpu().numpy(), ref["kv_list"]), "kv_list"
    assert np.array_equal(got["kv_count"][0].cpu().numpy(), ref["kv_count"]), "kv_count"
    return ref, got


def gpu_demand_pack(binding, shape, mask_d, rank_d, P, flags, Kd, Vd, ws, capacity_entries=None, dst_base=None):
    outs = binding.alloc_demand_outputs(shape, P)
    entry = 2 * shape.block * shape.head_dim * 2
    # plan first to size the buffer exactly
    binding.sparsp_demand_pack(shape, mask_d, rank_d, P, flags | binding.SPARSP_PLAN_ONLY, None, None,
                               outs["union_mask"], outs["cnt"], outs["seg_offset"], outs["seg_total"],
                               outs["volume_bytes"], None, 0, None, ws)
    torch.cuda.synchronize()
    total = int(outs["seg_total"].sum().item())
    n_ent = total if capacity_entries is None else capacity_entries
    packed = torch.full((max(n_ent * entry, 16) + 64,), 0xAB, dtype=torch.uint8, device="cuda")  # sentinel
    binding.sparsp_demand_pack(shape, mask_d, rank_d, P, flags, Kd, Vd, outs["union_mask"], outs["cnt"],
                               outs["seg_offset"], outs["seg_total"], outs["volume_bytes"], packed,
                               n_ent * entry, dst_base, ws)
    torch.cuda.synchronize()
    outs["packed"] = packed
    outs["total_entries"] = total
    return outs


def check_demand(oracle, binding, shape, mask_np, rank_np, P, include_local, got):
    ref = oracle.demand(mask_np, rank_np, P, shape.block, shape.head_dim, include_local=include_local)
    assert np.array_equal(u32(got["union_mask"][0]), ref["U"]), "union"
    assert np.array_equal(got["cnt"][0].cpu().numpy(), ref["cnt"]), "cnt"
    assert np.array_equal(got["seg_offset"][0].cpu().numpy(), ref["seg_off"]), "seg_offset"
    assert np.array_equal(got["seg_total"][0].cpu().numpy(), ref["total"]), "seg_total"
    assert np.array_equal(got["volume_bytes"][0].cpu().numpy(), ref["volume"]), "volume"
    return ref


def oracle_entry_list(ref, rank_np, P, H, NB, include_local):
    """(head, block) of every packed entry, in pack order, from the ORACLE's union words."""
    hs, js = [], []
    bit = np.arange(NB)
    for r in range(P):
        for p in range(P):
            if p == r and not include_local:
                continue
            for h in range(H):
                words = ref["U"][r, h]
                on = ((words[bit >> 5] >> (bit & 31).astype(np.uint32)) & 1).astype(bool) & (rank_np == p)
                jj = np.nonzero(on)[0]
                hs.append(np.full(len(jj), h, np.int64))
                js.append(jj.astype(np.int64))
    if not hs:
        return np.zeros(0, np.int64), np.zeros(0, np.int64)
    return np.concatenate(hs), np.concatenate(js)


def check_packed_full_on_device(Kd_hnd, Vd_hnd, b, packed, h_idx, j_idx):
    """Whole-buffer check in device memory: expected bytes = library gather (torch indexing) of the
    zero-padded block views of K and V by the oracle's entry list; trailing sentinel untouched."""
    H, N, d = Kd_hnd.shape
    NB = (N + b - 1) // b
    pad = NB * b - N
    Kp = torch.nn.functional.pad(Kd_hnd, (0, 0, 0, pad)).view(H, NB, b * d)
    Vp = torch.nn.functional.pad(Vd_hnd, (0, 0, 0, pad)).view(H, NB, b * d)
    hi = torch.as_tensor(h_idx, device=Kd_hnd.device)
    ji = torch.as_tensor(j_idx, device=Kd_hnd.device)
    n = len(h_idx)
    entry = 2 * b * d * 2
    got = packed[: n * entry].view(torch.bfloat16).view(n, 2, b * d)
    chunk = 4096
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        exp = torch.stack([Kp[hi[s:e], ji[s:e]], Vp[hi[s:e], ji[s:e]]], dim=1)
        assert torch.equal(got[s:e].view(torch.int16), exp.view(torch.int16)), f"packed entries {s}..{e}"
    assert bool((packed[n * entry:] == 0xAB).all()), "bytes beyond the last entry were written"


def sample_units(H, NB, rank_np, n_random, seed, extra_blocks=()):
    """Seeded sample of (head, query block) units: block 0, the last (ragged) block, one block per
    virtual rank, any extra blocks, plus random ones; heads rotate."""
    rng = np.random.default_rng(seed)
    blocks = [0, NB - 1] + [int(np.nonzero(rank_np == r)[0][0]) for r in np.unique(rank_np)] + list(extra_blocks)
    blocks += [int(x) for x in rng.integers(0, NB, n_random)]
    units = []
    for t, i in enumerate(blocks):
        units.append((int((t * 7 + int(rng.integers(0, H))) % H), i))
    return sorted(set(units))


def sample_units_per_head(H, NB, rank_np, n_random, seed, extra_blocks=(), full_heads=()):
    """Seeded sample that covers EVERY head: per head block 0, the last (ragged) block, the first block of
    every virtual rank, any extra blocks (e.g. the video/text boundary) and n_random random blocks drawn
    per head; the heads in `full_heads` contribute all their query blocks (with 64-token blocks the kernel
    stacks two query blocks per tile, so a fully covered head checks both members of every pair)."""
    rng = np.random.default_rng(seed)
    fixed = [0, NB - 1] + [int(np.nonzero(rank_np == r)[0][0]) for r in np.unique(rank_np)] + list(extra_blocks)
    units = []
    for h in range(H):
        if h in full_heads:
            blocks = range(NB)
        else:
            blocks = sorted(set(fixed + [int(x) for x in rng.integers(0, NB, n_random)]))
        units += [(h, int(i)) for i in blocks]
    return units


def check_attn_units(oracle, Q, K, V, mask_np, b, O_hnd_gpu, units, scale=None, lse_gpu=None, report=None):
    """O_hnd_gpu: device [H][N][d] bf16 view of the kernel's output.  The tolerance is asserted over the
    pooled sample and per head.  `report` (a dict) receives the figures: max / mean error, the reference
    value the maximum occurred at, and how much of the maximum is the rounding of the output to bf16."""
    ref, ref_lse = oracle.attn_rows(Q, K, V, mask_np, b, units, scale)
    H, N, d = Q.shape
    errs, per_head = [], {}
    worst = (-1.0, 0.0, 0.0)
    for u, (h, i) in enumerate(units):
        n_i = min(b, N - i * b)
        got = O_hnd_gpu[h, i * b:i * b + n_i].float().cpu().numpy()
        e = np.abs(got - ref[u, :n_i])
        errs.append(e.reshape(-1))
        per_head.setdefault(h, []).append(e.reshape(-1))
        if e.max() > worst[0]:
            idx = np.unravel_index(e.argmax(), e.shape)
            r = float(ref[u, :n_i][idx])
            rb = float(torch.tensor(r).to(torch.bfloat16).float())
            worst = (float(e.max()), r, abs(rb - r))
        if lse_gpu is not None:
            gl = lse_gpu[h, i * b:i * b + n_i].cpu().numpy()
            assert np.abs(gl - ref_lse[u, :n_i]).max() < 2e-2, ("lse", h, i)
    err = np.concatenate(errs)
    assert np.isfinite(err).all()
    assert err.max() <= ATTN_MAX_ABS, f"max abs err {err.max():.4g} at reference value {worst[1]:.4g}"
    assert err.mean() <= ATTN_MEAN_ABS, f"mean abs err {err.mean():.4g}"
    for h, es in per_head.items():
        eh = np.concatenate(es)
        assert eh.max() <= ATTN_MAX_ABS and eh.mean() <= ATTN_MEAN_ABS, f"head {h}: max {eh.max():.4g} mean {eh.mean():.4g}"
    if report is not None:
        report.update(units=len(units), max_abs=float(err.max()), mean_abs=float(err.mean()), ref_at_max=worst[1],
                      bf16_rounding_of_ref_at_max=worst[2],
                      worst_head_mean=float(max(np.concatenate(es).mean() for es in per_head.values())))
    return float(err.max()), float(err.mean())
