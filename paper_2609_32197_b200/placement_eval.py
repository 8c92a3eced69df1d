"""Compares block placements on a workload: exchange volume (Eq. "sparse-exchange-volume") and how widely
received K blocks are shared by the receiving rank's queries (Section 3.2), for contiguous, interval-periodic
(Eq. "periodic-placement") and shuffled layouts, across virtual rank counts and sparsity levels; also times
the token permutation that applies a layout.  Everything runs through the C-ABI calls on the GPU.

    python -m paper_2609_32197_b200.placement_eval --workload wan [--ranks 2 4 8] [--pct 5 10 25] [--tau 0.9]
"""
from __future__ import annotations

import argparse

import torch

from . import binding, synth


def _rank(shape, NB, P, name):
    if name == "contiguous":
        return binding.sparsp_placement_contiguous(shape, P)
    if name == "periodic":
        return binding.sparsp_placement_periodic(shape, P)
    return synth.shuffled_placement(NB, P, seed=1)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="mid", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--ranks", type=int, nargs="+", default=[2, 4, 8])
    ap.add_argument("--pct", type=int, nargs="+", default=None, help="top-k levels in percent of the video blocks")
    ap.add_argument("--tau", type=float, nargs="+", default=None, help="CDF thresholds instead of top-k levels")
    ap.add_argument("--band", type=int, nargs="+", default=None,
                    help="instead of masks from the synthetic Q/K: the multi-diagonal demand model of Section 4.3, every "
                         "query block keeps the blocks within this many in-frame positions of its own, in every frame")
    ap.add_argument("--heads", type=int, default=0)
    args = ap.parse_args(argv)
    wl0 = synth.WORKLOADS[args.workload]
    wl = wl0 if not args.heads else synth.Workload(wl0.name, args.heads, wl0.head_dim, wl0.grid, wl0.n_text, wl0.block,
                                                   wl0.topk_abs, wl0.topk_pct, wl0.ranks)
    H, d, b = wl.heads, wl.head_dim, wl.block
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    g = binding.sparsp_geometry(shape)
    NB = g.n_blocks
    Q, K, V = synth.make_qkv(wl, "cuda")
    ws = binding.make_workspace(shape, max(args.ranks))
    if args.band:
        levels = [("band", dlt) for dlt in args.band]
    elif args.tau:
        levels = [("tau", t) for t in args.tau]
    elif args.pct:
        levels = [("pct", p) for p in args.pct]
    else:
        levels = [("k", wl.topk_abs)] if wl.topk_abs else [("pct", p) for p in wl.topk_pct]
    mask = torch.zeros(1, H, NB, g.n_words, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, H, NB, dtype=torch.int32, device="cuda")
    print(f"workload {wl.name}: {g.n_tokens} tokens, {NB} blocks of {b}, {H} heads")
    print("| selection | kept/row | ranks | placement | volume GB | vs contiguous | remote blocks shared by >= 10 / 25 / 50 % of the local queries |")
    print("|---|---|---|---|---|---|---|")
    for kind, val in levels:
        if kind == "band":
            import numpy as np
            F = wl.grid[1] * wl.grid[2]
            first = np.arange(NB, dtype=np.int64) * b
            pos = np.where(first < wl.n_video, (first % F) // b, -1)          # in-frame block position; -1 = text
            keep = (np.abs(pos[:, None] - pos[None, :]) <= val) | (pos[:, None] < 0) | (pos[None, :] < 0)
            words = np.zeros((NB, g.n_words), np.uint32)
            for j in range(NB):
                words[:, j >> 5] |= keep[:, j].astype(np.uint32) << np.uint32(j & 31)
            mask.copy_(torch.as_tensor(np.broadcast_to(words, (1, H, NB, g.n_words)).copy().view(np.int32)))
            cnt.copy_(torch.as_tensor(np.broadcast_to(keep.sum(1).astype(np.int32), (1, H, NB)).copy()))
            label = f"band {val}"
        elif kind == "tau":
            binding.sparsp_block_mask_cdf(shape, Q, K, val, 0.0, mask, cnt, None, None, ws)
            label = f"cdf {val:g}"
        else:
            k = val if kind == "k" else binding.sparsp_resolve_topk(val, g.n_video_blocks)
            binding.sparsp_block_mask(shape, Q, K, k, mask, None, cnt, None, None, ws)
            label = f"top-{k}"
        kept = cnt.float().mean().item()
        for P in args.ranks:
            do = binding.alloc_demand_outputs(shape, P)
            base = None
            for name in ("contiguous", "periodic", "shuffle"):
                rank_d = _rank(shape, NB, P, name).cuda()
                binding.sparsp_demand_pack(shape, mask, rank_d, P, binding.SPARSP_PLAN_ONLY, None, None, do["union_mask"],
                                           do["cnt"], do["seg_offset"], do["seg_total"], do["volume_bytes"], None, 0, None, ws)
                hist = torch.zeros(1, P, 101, dtype=torch.int64, device="cuda")
                binding.sparsp_sharing_histogram(shape, mask, rank_d, P, hist)
                vol = do["volume_bytes"].sum().item()
                base = vol if base is None else base
                hsum = hist[0].sum(0).double()
                tot = max(hsum.sum().item(), 1.0)
                ge = [hsum[x:].sum().item() / tot for x in (10, 25, 50)]
                print(f"| {label} | {kept:.1f} | {P} | {name} | {vol / 1e9:.3f} | {vol / base - 1:+.1%} | "
                      f"{ge[0]:.1%} / {ge[1]:.1%} / {ge[2]:.1%} |")
    # the permutation that applies a layout: one read + one write of the tensor
    P = wl.ranks
    bos, off, _ = binding.sparsp_placement_permutation(shape, P, _rank(shape, NB, P, "periodic"))
    bos_d, off_d = bos.cuda(), off.cuda()
    Y = torch.empty_like(Q)
    for _ in range(3):
        binding.sparsp_permute_tokens(shape, Q, Y, bos_d, off_d, False)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(10):
        binding.sparsp_permute_tokens(shape, Q, Y, bos_d, off_d, False)
        binding.sparsp_permute_tokens(shape, Y, Q, bos_d, off_d, True)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 20
    print(f"token permutation ({P} ranks, periodic): {ms:.3f} ms per tensor, {2 * Q.numel() * 2 / ms / 1e6:.0f} GB/s (read + write)")


if __name__ == "__main__":
    main()
