#!/usr/bin/env python
"""Benchmark of the SparSP single-device hot path on B200.

One *step* = one attention layer's worth of the whole path on one batch of synthetic inputs:
    sparsp_block_mask  ->  sparsp_demand_pack  ->  sparsp_sparse_attn_fwd
Prints ONE JSON line (rank 0).  `value` = kept-block attention FLOPs of all ranks / step time, i.e.
effective TFLOP/s of the whole layer; the per-kernel figures (attention TFLOP/s against the bf16
tensor peak, pack GB/s against the HBM copy peak, ms per stage) ride along in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mid|cog|wan|hunyuan|tiny]
                    [--pct P] [--placement contiguous|periodic|shuffle] [--impl ours|reference]

With N > 1 launch under torch.distributed.run; every rank runs its own replica of the workload
(different seed) -- the path has no exchange step on one node, so scaling is weak and there is no
data-path collective.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sparse-attn effective TFLOP/s + %bf16 peak; pack GB/s + %HBM; ms/layer"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the attention kernel, from the ncu
# captures summarised under profiles/ (None = not captured for that workload).
ATTN_DRAM_TRAFFIC = {
    ("mid", 58): 591.0e6,            # profiles/attn_fwd_kernel_mid_and_hunyuan4.md, full workload
    ("hunyuan", 93): 6 * 710.0e6,     # same file: 4-head capture scaled by heads (24 / 4)
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.05):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
            "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
            "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
            "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap,
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def resolve_workload(args):
    from paper_2609_32197_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    if args.heads:
        wl = synth.Workload(wl.name, args.heads, wl.head_dim, wl.grid, wl.n_text, wl.block, wl.topk_abs,
                            wl.topk_pct, wl.ranks, wl.placements, seed=wl.seed)
    placement = args.placement or wl.placements[0]
    return wl, placement


def kept_flops_and_counts(mask_i32, N, b, d):
    """4*d*sum over kept (h,i,j) of rows_i*cols_j, from the device mask (library tensor ops)."""
    import torch
    B, H, NB, Wd = mask_i32.shape
    bits = torch.arange(32, device=mask_i32.device, dtype=torch.int32)
    m = ((mask_i32.unsqueeze(-1) >> bits) & 1).reshape(B, H, NB, Wd * 32)[..., :NB].to(torch.float64)
    sizes = torch.full((NB,), float(b), dtype=torch.float64, device=mask_i32.device)
    sizes[-1] = float(N - (NB - 1) * b)
    pairs = torch.einsum("i,bhij,j->", sizes, m, sizes).item()
    return 4.0 * d * pairs, int(m.sum().item())


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_32197_b200 import binding, dist_util, synth

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    wl, placement = resolve_workload(args)
    wl = dist_util.replica_workload(wl, rank)  # every rank its own replica of the workload
    H, d, b, P = wl.heads, wl.head_dim, wl.block, wl.ranks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    g = binding.sparsp_geometry(shape)
    N, NB = g.n_tokens, g.n_blocks
    pct = args.pct if args.pct else (wl.topk_pct[0] if wl.topk_pct else None)
    k = wl.topk_abs if pct is None else binding.sparsp_resolve_topk(pct, g.n_video_blocks)

    Q, K, V = synth.make_qkv(wl, dev)
    if placement == "contiguous":
        rank_of_block = binding.sparsp_placement_contiguous(shape, P)
    elif placement == "periodic":
        rank_of_block = binding.sparsp_placement_periodic(shape, P)
    else:
        rank_of_block = synth.shuffled_placement(NB, P, seed=1)
    rank_d = rank_of_block.to(dev)

    ws = binding.make_workspace(shape, P, dev)
    mo = binding.alloc_mask_outputs(shape, k, dev, with_list=True)
    do = binding.alloc_demand_outputs(shape, P, dev)
    O = torch.empty_like(Q)
    entry = 2 * b * d * 2

    def step_mask():
        if args.tau > 0:  # CDF-threshold selection instead of top-k (rows keep different numbers of blocks)
            binding.sparsp_block_mask_cdf(shape, Q, K, args.tau, 0.0, mo["mask"], mo["kv_count"], None, None, ws)
        else:
            binding.sparsp_block_mask(shape, Q, K, k, mo["mask"], mo["kv_list"], mo["kv_count"], None, None, ws)

    def step_plan():
        binding.sparsp_demand_pack(shape, mo["mask"], rank_d, P, binding.SPARSP_PLAN_ONLY, None, None,
                                   do["union_mask"], do["cnt"], do["seg_offset"], do["seg_total"],
                                   do["volume_bytes"], None, 0, None, ws)

    # size the packed buffer once (the mask is a function of the inputs, which do not change)
    step_mask()
    step_plan()
    torch.cuda.synchronize()
    total_entries = int(do["seg_total"].sum().item())
    packed = torch.empty(max(total_entries * entry, 16), dtype=torch.uint8, device=dev)
    volume = do["volume_bytes"].sum().item()

    def step_pack():
        binding.sparsp_demand_pack(shape, mo["mask"], rank_d, P, 0, K, V, do["union_mask"], do["cnt"],
                                   do["seg_offset"], do["seg_total"], do["volume_bytes"], packed,
                                   packed.numel(), None, ws)

    def step_attn():
        binding.sparsp_sparse_attn_fwd(shape, Q, K, V, mo["mask"], 0.0, O, None, ws)

    def step():
        step_mask()
        step_pack()
        step_attn()

    flops, kept_pairs = kept_flops_and_counts(mo["mask"], N, b, d)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    launches0 = binding.sparsp_launch_count()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    barrier()
    for s in range(args.steps):
        ev[s][0].record(stream)
        step_mask()
        ev[s][1].record(stream)
        step_pack()
        ev[s][2].record(stream)
        step_attn()
        ev[s][3].record(stream)
    end = torch.cuda.Event(enable_timing=True)
    end.record(stream)
    barrier()
    launches = binding.sparsp_launch_count() - launches0
    total_ms = ev[0][0].elapsed_time(end)
    clocks = sampler.finish()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()

    def avg(i):
        return sum(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(args.steps)) / args.steps

    mask_ms, dpack_ms, attn_ms = avg(0), avg(1), avg(2)

    # demand bookkeeping alone (plan-only call), to separate the gather kernel's time
    pe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    step_plan()
    torch.cuda.synchronize()
    pe[0].record(stream)
    for _ in range(args.steps):
        step_plan()
    pe[1].record(stream)
    torch.cuda.synchronize()
    plan_ms = pe[0].elapsed_time(pe[1]) / args.steps
    pack_ms = max(dpack_ms - plan_ms, 1e-6)

    # End to end through the public API from pinned host buffers, result read back to the host.  The path is
    # independent per head, so the heads go through in a few chunks on three streams (copy in, compute, copy
    # out): a chunk's kernels run while the next chunk's inputs arrive and the previous chunk's output leaves.
    h2d = 3 * Q.numel() * 2
    d2h = O.numel() * 2 + do["volume_bytes"].numel() * 8
    e2e_ms = float("nan")
    e2e_chunks = 0
    if not args.no_e2e:
        hQ, hK, hV = (torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in (Q, K, V))
        hQ.copy_(Q); hK.copy_(K); hV.copy_(V)
        hO = torch.empty(O.shape, dtype=O.dtype, pin_memory=True)
        n_chunks = min(4, H) if h2d >= (32 << 20) else 1  # a small workload gains nothing from more launches
        e2e_chunks = n_chunks
        bounds = [(c * H // n_chunks, (c + 1) * H // n_chunks) for c in range(n_chunks)]
        chunks = []
        for (h0, h1) in bounds:
            sh = binding.make_shape(h1 - h0, d, wl.grid, wl.n_text, b)
            c = {"h": (h0, h1), "shape": sh, "ws": binding.make_workspace(sh, P, dev),
                 "mo": binding.alloc_mask_outputs(sh, k, dev, with_list=True),
                 "do": binding.alloc_demand_outputs(sh, P, dev)}
            c["hVol"] = torch.empty(c["do"]["volume_bytes"].shape, dtype=torch.int64, pin_memory=True)
            chunks.append(c)

        def chunk_mask(c):
            h0, h1 = c["h"]
            if args.tau > 0:
                binding.sparsp_block_mask_cdf(c["shape"], Q[h0:h1], K[h0:h1], args.tau, 0.0, c["mo"]["mask"],
                                              c["mo"]["kv_count"], None, None, c["ws"])
            else:
                binding.sparsp_block_mask(c["shape"], Q[h0:h1], K[h0:h1], k, c["mo"]["mask"], c["mo"]["kv_list"],
                                          c["mo"]["kv_count"], None, None, c["ws"])

        def chunk_pack(c, plan_only):
            h0, h1 = c["h"]
            o = c["do"]
            binding.sparsp_demand_pack(c["shape"], c["mo"]["mask"], rank_d, P,
                                       binding.SPARSP_PLAN_ONLY if plan_only else 0,
                                       None if plan_only else K[h0:h1], None if plan_only else V[h0:h1],
                                       o["union_mask"], o["cnt"], o["seg_offset"], o["seg_total"], o["volume_bytes"],
                                       None if plan_only else c["packed"], 0 if plan_only else c["packed"].numel(),
                                       None, c["ws"])

        for c in chunks:  # size each chunk's packed buffer once (the masks are a function of the inputs)
            chunk_mask(c)
            chunk_pack(c, True)
            torch.cuda.synchronize()
            c["packed"] = torch.empty(max(int(c["do"]["seg_total"].sum().item()) * entry, 16), dtype=torch.uint8,
                                      device=dev)
        s_in, s_comp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev_in = [torch.cuda.Event() for _ in chunks]
        ev_comp = [torch.cuda.Event() for _ in chunks]
        ev_out = [torch.cuda.Event() for _ in chunks]

        def e2e_step():
            for i, c in enumerate(chunks):
                h0, h1 = c["h"]
                with torch.cuda.stream(s_in):
                    s_in.wait_event(ev_comp[i])  # the previous step's kernels have read this slice
                    Q[h0:h1].copy_(hQ[h0:h1], non_blocking=True)
                    K[h0:h1].copy_(hK[h0:h1], non_blocking=True)
                    V[h0:h1].copy_(hV[h0:h1], non_blocking=True)
                    ev_in[i].record(s_in)
                with torch.cuda.stream(s_comp):
                    s_comp.wait_event(ev_in[i])
                    s_comp.wait_event(ev_out[i])  # the previous step's output slice has left
                    chunk_mask(c)
                    chunk_pack(c, False)
                    binding.sparsp_sparse_attn_fwd(c["shape"], Q[h0:h1], K[h0:h1], V[h0:h1], c["mo"]["mask"], 0.0,
                                                   O[h0:h1], None, c["ws"])
                    ev_comp[i].record(s_comp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[i])
                    hO[h0:h1].copy_(O[h0:h1], non_blocking=True)
                    c["hVol"].copy_(c["do"]["volume_bytes"], non_blocking=True)
                    ev_out[i].record(s_out)

        def join():
            for st_ in (s_in, s_comp, s_out):
                stream.wait_stream(st_)

        e2e_steps = max(1, min(args.steps, 5))
        for st_ in (s_in, s_comp, s_out):
            st_.wait_stream(stream)
        e2e_step()
        join()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for st_ in (s_in, s_comp, s_out):
            st_.wait_stream(stream)
        for _ in range(e2e_steps):
            e2e_step()
        join()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        assert all(binding.sparsp_status(c["ws"]) == binding.SPARSP_OK for c in chunks)
        assert int(sum(int(c["hVol"].sum().item()) for c in chunks)) == int(volume)

    # max over ranks (device-timed), whole-job totals
    tm, tot = dist_util.reduce_over_ranks(
        {"total": total_ms, "e2e": e2e_ms if e2e_ms == e2e_ms else 0.0, "attn": attn_ms, "pack": pack_ms, "mask": mask_ms},
        {"flops": flops, "launches": float(launches)}, dev)
    total_ms, attn_ms, pack_ms, mask_ms = tm["total"], tm["attn"], tm["pack"], tm["mask"]
    if e2e_ms == e2e_ms:
        e2e_ms = tm["e2e"]
    flops_all, launches_all = tot["flops"], tot["launches"]
    ms_per_step = total_ms / args.steps

    peaks = load_peaks()
    attn_tflops = flops / (attn_ms * 1e-3) / 1e12
    pack_bytes = 2.0 * volume
    pack_gbs = pack_bytes / (pack_ms * 1e-3) / 1e9 if volume else 0.0
    result = {
        "metric": METRIC,
        "value": flops_all / (ms_per_step * 1e-3) / 1e12,
        "unit": "TFLOP/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": ms_per_step,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16",
        "data": "synthetic",
        "config": {
            "workload": wl.name, "heads": H, "head_dim": d, "grid": list(wl.grid), "n_text": wl.n_text,
            "tokens": N, "block": b, "n_blocks": NB, "topk_blocks": (k if args.tau <= 0 else None),
            "selection": ("top-k" if args.tau <= 0 else "cdf tau=%g" % args.tau), "kept_pairs": kept_pairs,
            "virtual_ranks": P, "placement": placement, "layout": "[H][N][d]",
            "l2_policy": "inputs larger than L2 (Q+K+V = %.0f MB)" % (3 * Q.numel() * 2 / 1e6),
        },
        "ms_per_layer": ms_per_step,
        "stage_ms": {"block_mask": mask_ms, "demand_plan": plan_ms, "pack": pack_ms, "sparse_attn": attn_ms},
        "attn_tflops": attn_tflops,
        "attn_pct_bf16_peak": {"of_measured_burst": attn_tflops / peaks["bf16_tflops"],
                               "of_measured_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                               "of_nominal": attn_tflops / NOMINAL["bf16_tflops"]},
        "pack_gbs": pack_gbs,
        "pack_pct_hbm": {"of_measured": pack_gbs / peaks["hbm_gbs"], "of_nominal": pack_gbs / NOMINAL["hbm_gbs"]},
        "volume_bytes_total": volume,
        "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel (+ attn_prep_kernel, timed together)", "achieved": attn_tflops,
                     "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " burst", "unit": "TFLOP/s",
                     "frac": attn_tflops / peaks["bf16_tflops"],
                     "traffic": ATTN_DRAM_TRAFFIC.get((wl.name, k)) if args.tau <= 0 else None},
        "roofline_pack": {"bound": "hbm", "kernel": "pack_bulk_kernel", "achieved": pack_gbs, "peak": peaks["hbm_gbs"],
                          "peak_source": peaks["source"], "unit": "GB/s", "frac": pack_gbs / peaks["hbm_gbs"],
                          "algorithmic_bytes": pack_bytes},
        "e2e": {"value": None if e2e_ms != e2e_ms else flops_all / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                "ms_per_step": None if e2e_ms != e2e_ms else e2e_ms, "head_chunks": e2e_chunks,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches_all),
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl, k, placement, rank_of_block.numpy(), Q, K, V, flops, budget_s=15.0)
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# CPU baseline / reference arm: the oracle as it stands, on a bounded sample
# ------------------------------------------------------------------------------------------------
def oracle_sample_time(wl, k, rank_np, Qh, Kh, Vh, n_units):
    """Times the oracle on ONE head for steps 1-2 and on n_units (head 0, query block) units for
    step 3.  Returns the seconds of each part and the kept flops of the sampled attention units."""
    import numpy as np

    import oracle
    b, d, P = wl.block, wl.head_dim, wl.ranks
    N = Qh.shape[1]
    t0 = time.perf_counter()
    ref = oracle.block_mask(Qh, Kh, b, k, wl.n_text)
    t1 = time.perf_counter()
    dref = oracle.demand(ref["mask"], rank_np, P, b, d)
    oracle.pack(Kh, Vh, dref["U"], rank_np, b, P, dref["total"])
    t2 = time.perf_counter()
    NB = ref["mask"].shape[1]
    rng = np.random.default_rng(0)
    if n_units >= NB:
        blocks = list(range(NB))
    else:
        blocks = sorted(set([0, NB - 1] + [int(x) for x in rng.integers(0, NB, max(n_units - 2, 0))]))
    units = [(0, i) for i in blocks]
    t3 = time.perf_counter()
    oracle.attn_rows(Qh, Kh, Vh, ref["mask"], b, units)
    t4 = time.perf_counter()
    sizes = np.full(NB, b, np.float64)
    sizes[-1] = N - (NB - 1) * b
    fl = 0.0
    for (_, i) in units:
        row = ref["mask"][0, i]
        on = np.array([(int(row[j >> 5]) >> (j & 31)) & 1 for j in range(NB)], np.float64)
        fl += 4.0 * d * sizes[i] * float((on * sizes).sum())
    return dict(mask_s=t1 - t0, pack_s=t2 - t1, attn_s=t4 - t3, attn_flops=fl, n_units=len(units))


def cpu_baseline(wl, k, placement, rank_np, Q, K, V, layer_flops, budget_s=15.0):
    """The oracle, as it stands, on the host cores: whole heads (steps 1-2 in full, step 3 on as many of the
    head's query blocks as the time left allows) until about budget_s seconds are spent."""
    import oracle
    oracle.build()
    H, NB = wl.heads, wl.n_blocks
    Qh, Kh, Vh = (x[:1].cpu() for x in (Q, K, V))
    probe = oracle_sample_time(wl, k, rank_np, Qh, Kh, Vh, 2)
    per_unit = probe["attn_s"] / probe["n_units"]
    acc = dict(mask_s=0.0, pack_s=0.0, attn_s=0.0, attn_flops=0.0, n_units=0, heads=0)
    t_start = time.perf_counter()
    for h in range(H):
        left = budget_s - (time.perf_counter() - t_start)
        if h > 0 and left < 0.05 * budget_s:
            break
        n_units = int(max(2, min(NB, left / max(per_unit, 1e-6))))
        Qh, Kh, Vh = (x[h:h + 1].cpu() for x in (Q, K, V))
        s = oracle_sample_time(wl, k, rank_np, Qh, Kh, Vh, n_units)
        for key in ("mask_s", "pack_s", "attn_s", "attn_flops", "n_units"):
            acc[key] += s[key]
        acc["heads"] += 1
        per_unit = acc["attn_s"] / acc["n_units"]
    hs = acc["heads"]
    layer_s = H * (acc["mask_s"] + acc["pack_s"]) / hs + acc["attn_s"] * (layer_flops / max(acc["attn_flops"], 1.0))
    return {"value": layer_flops / layer_s / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "steps 1-2 on %d of %d heads (scaled to %d), step 3 on %d (head, query block) units of those "
                      "heads scaled by kept flops; %.1f s measured, extrapolated layer time %.1f s"
                      % (hs, H, H, acc["n_units"], acc["mask_s"] + acc["pack_s"] + acc["attn_s"], layer_s),
            "measured_s": {"mask": acc["mask_s"], "demand_pack": acc["pack_s"], "attn_sample": acc["attn_s"]}}


def run_reference(args):
    """Reference arm for this build = the CPU oracle, unmodified, on the host cores."""
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if rank != 0:
        return
    import numpy as np
    import torch

    import oracle
    from paper_2609_32197_b200 import synth
    oracle.build()
    wl, placement = resolve_workload(args)
    H, d, b, P = wl.heads, wl.head_dim, wl.block, wl.ranks
    pct = args.pct if args.pct else (wl.topk_pct[0] if wl.topk_pct else None)
    k = wl.topk_abs if pct is None else oracle.resolve_topk(pct, wl.nb_video)
    NB = wl.n_blocks
    if placement == "contiguous":
        rank_np = oracle.placement_contiguous(NB, P)
    elif placement == "periodic":
        rank_np = oracle.placement_periodic(NB, P, b, wl.frame_tokens, wl.n_video)
    else:
        rank_np = synth.shuffled_placement(NB, P, seed=1).numpy()
    Qh, Kh, Vh = synth.make_qkv(wl, "cpu", heads=1)
    n_units = 4
    times, flops_s = [], []
    for it in range(args.warmup + args.steps):
        s = oracle_sample_time(wl, k, rank_np, Qh, Kh, Vh, n_units)
        if it >= args.warmup:
            times.append(s["mask_s"] + s["pack_s"] + s["attn_s"])
            # layer throughput extrapolated from the sample: flops of the sampled units over the
            # time the sample's share of the layer took
            frac_units = s["n_units"] / NB  # of one head's query blocks
            sample_s = (s["mask_s"] + s["pack_s"]) * frac_units + s["attn_s"]
            flops_s.append(s["attn_flops"] / sample_s)
    value = float(np.mean(flops_s)) / 1e12
    ms = 1e3 * float(np.mean(times))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "heads": H, "head_dim": d, "grid": list(wl.grid), "n_text": wl.n_text,
                   "tokens": wl.n_tokens, "block": b, "n_blocks": NB, "topk_blocks": k, "virtual_ranks": P,
                   "placement": placement, "layout": "[H][N][d]"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "each step: steps 1-2 on 1 head, step 3 on %d query blocks of that head; "
                                   "throughput = sampled kept flops / (sample's share of steps 1-2 + step 3 time)"
                                   % n_units},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mid", choices=["tiny", "mid", "cog", "wan", "hunyuan"])
    ap.add_argument("--pct", type=int, default=0, help="top-k as a percentage of the video blocks")
    ap.add_argument("--tau", type=float, default=0.0, help="CDF-threshold selection with this mass instead of top-k (ours only)")
    ap.add_argument("--placement", default=None, choices=[None, "contiguous", "periodic", "shuffle"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--heads", type=int, default=0, help="override the head count (small profiling cases)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
