#!/usr/bin/env python
"""Benchmark of the SparSP single-device hot path on B200.

One *step* = one attention layer's worth of the whole path on one batch of synthetic inputs:
    sparsp_block_mask  ->  sparsp_demand_pack  ->  sparsp_sparse_attn_fwd
Prints ONE JSON line (rank 0).  `value` = kept-block attention FLOPs of all ranks / step time, i.e.
effective TFLOP/s of the whole layer; the per-kernel figures (attention TFLOP/s against the bf16
tensor peak, pack GB/s against the HBM copy peak, ms per stage) ride along in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload hunyuan|wan|cog|mid|tiny]
                    [--pct P] [--placement contiguous|periodic|shuffle] [--impl ours|reference]
                    [--shard replicas|heads] [--no-per-config] [--sustained-s S] [--no-graph]

The headline configuration is the largest single-GPU one (Hunyuan-like, 118 800 tokens, top-k 10 %); at
N = 1 the same line carries `per_config` (all eight configurations of the contract measured the same way)
and `sustained` (the attention call alone, back to back for a couple of seconds, with the clocks sampled);
`graph_ms_per_step` is the same step captured once in a CUDA graph and replayed (the headline stays plain launches).
With N > 1 launch under torch.distributed.run; every rank runs its own replica of the workload
(different seed; weak scaling) or, with --shard heads, its share of the heads of ONE layer (strong
scaling) -- either way the path has no exchange step, so there is no data-path collective.
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
L2_BYTES = 126 << 20
# the configurations of the per_config list: (workload, top-k percent or None, placement)
PER_CONFIG = [("tiny", None, "contiguous"), ("mid", 15, "contiguous"), ("cog", 20, "shuffle"),
              ("wan", 10, "contiguous"), ("wan", 10, "periodic"),
              ("hunyuan", 5, "contiguous"), ("hunyuan", 10, "contiguous"), ("hunyuan", 25, "contiguous")]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def load_attn_traffic():
    """DRAM bytes per launch of the attention kernel from the ncu captures summarised under profiles/
    (dram__bytes_read.sum + dram__bytes_write.sum).  The table is a text file: one line per capture,
    `workload topk_blocks heads_captured bytes source`; a capture of fewer heads than the workload has is
    scaled by the head ratio (traffic grows in proportion to the heads: every head has its own Q, K, V, O).
    Returns {(workload, topk): (bytes_per_full_launch, note)}."""
    table = {}
    path = os.path.join(ROOT, "profiles", "attn_dram_traffic.txt")
    if not os.path.exists(path):
        return table
    from paper_2609_32197_b200 import synth
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            name, k, heads, nbytes, source = line.split(None, 4)
            full = synth.WORKLOADS[name].heads
            table[(name, int(k))] = (float(nbytes) * full / int(heads),
                                     "ncu capture of %s of %d heads (%s), not measured in this run" % (heads, full, source))
    return table


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
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


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


def describe_config(wl, heads, k, tau, kept_pairs, placement):
    """The `config` object of a result line (the same keys and values in both arms)."""
    input_bytes = 3 * heads * wl.n_tokens * wl.head_dim * 2
    if input_bytes >= 2 * L2_BYTES:
        l2 = "inputs larger than L2 (Q+K+V = %.0f MB)" % (input_bytes / 1e6)
    else:
        l2 = "L2 flushed between iterations (a %d MB buffer is overwritten; Q+K+V = %.1f MB)" % (
            (2 * L2_BYTES) >> 20, input_bytes / 1e6)
    return {"workload": wl.name, "heads": heads, "head_dim": wl.head_dim, "grid": list(wl.grid), "n_text": wl.n_text,
            "tokens": wl.n_tokens, "block": wl.block, "n_blocks": wl.n_blocks, "topk_blocks": (k if tau <= 0 else None),
            "selection": ("top-k" if tau <= 0 else "cdf tau=%g" % tau), "kept_pairs": kept_pairs,
            "virtual_ranks": wl.ranks, "placement": placement, "layout": "[H][N][d]", "l2_policy": l2}


def kept_flops_and_counts(mask_i32, N, b, d):
    """4*d*sum over kept (h,i,j) of rows_i*cols_j, from the device mask (library tensor ops)."""
    import torch
    B, H, NB, Wd = mask_i32.shape
    bits = torch.arange(32, device=mask_i32.device, dtype=torch.int32)
    sizes = torch.full((NB,), float(b), dtype=torch.float64, device=mask_i32.device)
    sizes[-1] = float(N - (NB - 1) * b)
    pairs, kept = 0.0, 0
    for h in range(H):  # head by head: the unpacked mask of a whole layer would be gigabytes
        m = ((mask_i32[:, h].unsqueeze(-1) >> bits) & 1).reshape(B, NB, Wd * 32)[..., :NB].to(torch.float64)
        pairs += torch.einsum("i,bij,j->", sizes, m, sizes).item()
        kept += int(m.sum().item())
    return 4.0 * d * pairs, kept


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
class Config:
    """One workload resident on the device with its buffers and the three calls of a step."""

    def __init__(self, wl, placement, pct, tau, dev, head_range=None):
        import torch

        from paper_2609_32197_b200 import binding, synth
        self.binding, self.wl, self.placement, self.tau, self.dev = binding, wl, placement, tau, dev
        h0, h1 = head_range if head_range else (0, wl.heads)
        self.H, self.d, self.b, self.P = h1 - h0, wl.head_dim, wl.block, wl.ranks
        self.shape = binding.make_shape(self.H, self.d, wl.grid, wl.n_text, self.b)
        g = binding.sparsp_geometry(self.shape)
        self.N, self.NB = g.n_tokens, g.n_blocks
        self.k = wl.topk_abs if pct is None else binding.sparsp_resolve_topk(pct, g.n_video_blocks)
        self.Q, self.K, self.V = synth.make_qkv(wl, dev, heads=self.H, head_begin=h0)
        if placement == "contiguous":
            self.rank_of_block = binding.sparsp_placement_contiguous(self.shape, self.P)
        elif placement == "periodic":
            self.rank_of_block = binding.sparsp_placement_periodic(self.shape, self.P)
        else:
            self.rank_of_block = synth.shuffled_placement(self.NB, self.P, seed=1)
        self.rank_d = self.rank_of_block.to(dev)
        self.ws = binding.make_workspace(self.shape, self.P, dev)
        self.mo = binding.alloc_mask_outputs(self.shape, self.k, dev, with_list=True)
        self.do = binding.alloc_demand_outputs(self.shape, self.P, dev)
        self.O = torch.empty_like(self.Q)
        self.entry = 2 * self.b * self.d * 2
        # size the packed buffer once (the mask is a function of the inputs, which do not change)
        self.step_mask()
        self.step_plan()
        torch.cuda.synchronize()
        total_entries = int(self.do["seg_total"].sum().item())
        self.packed = torch.empty(max(total_entries * self.entry, 16), dtype=torch.uint8, device=dev)
        self.volume = int(self.do["volume_bytes"].sum().item())
        self.flops, self.kept_pairs = kept_flops_and_counts(self.mo["mask"], self.N, self.b, self.d)
        self.input_bytes = 3 * self.Q.numel() * 2
        # a working set that fits L2 would turn "HBM GB/s" into an L2 figure: flush L2 between iterations
        self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if self.input_bytes < 2 * L2_BYTES else None

    def step_mask(self):
        b, mo = self.binding, self.mo
        if self.tau > 0:  # CDF-threshold selection instead of top-k (rows keep different numbers of blocks)
            b.sparsp_block_mask_cdf(self.shape, self.Q, self.K, self.tau, 0.0, mo["mask"], mo["kv_count"], None, None, self.ws)
        else:
            b.sparsp_block_mask(self.shape, self.Q, self.K, self.k, mo["mask"], mo["kv_list"], mo["kv_count"], None, None,
                                self.ws)

    def step_plan(self):
        b, do = self.binding, self.do
        b.sparsp_demand_pack(self.shape, self.mo["mask"], self.rank_d, self.P, b.SPARSP_PLAN_ONLY, None, None,
                             do["union_mask"], do["cnt"], do["seg_offset"], do["seg_total"], do["volume_bytes"], None, 0,
                             None, self.ws)

    def step_pack(self):
        b, do = self.binding, self.do
        b.sparsp_demand_pack(self.shape, self.mo["mask"], self.rank_d, self.P, 0, self.K, self.V, do["union_mask"],
                             do["cnt"], do["seg_offset"], do["seg_total"], do["volume_bytes"], self.packed,
                             self.packed.numel(), None, self.ws)

    def step_attn(self):
        self.binding.sparsp_sparse_attn_fwd(self.shape, self.Q, self.K, self.V, self.mo["mask"], 0.0, self.O, None, self.ws)

    def step(self):
        self.step_mask()
        self.step_pack()
        self.step_attn()

    def check_status(self):
        assert self.binding.sparsp_status(self.ws) == self.binding.SPARSP_OK, self.binding.sparsp_last_error()

    def describe(self):
        return describe_config(self.wl, self.H, self.k, self.tau, self.kept_pairs, self.placement)


def time_steps(cfg, steps, warmup, barrier, local_gpu):
    """W warm-up steps, then `steps` timed steps bracketed by `barrier`; per-stage CUDA events on the launching
    stream.  Returns the device times (ms), the launch count and the clocks sampled during the timed region."""
    import torch
    binding = cfg.binding
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        cfg.step()
    barrier()
    cfg.check_status()
    sampler = ClockSampler(physical_gpu_index(local_gpu))
    sampler.start()
    launches0 = binding.sparsp_launch_count()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    barrier()
    for s in range(steps):
        if cfg.flush is not None:
            cfg.flush.fill_(s & 0xFF)
        ev[s][0].record(stream)
        cfg.step_mask()
        ev[s][1].record(stream)
        cfg.step_pack()
        ev[s][2].record(stream)
        cfg.step_attn()
        ev[s][3].record(stream)
    end = torch.cuda.Event(enable_timing=True)
    end.record(stream)
    barrier()
    launches = binding.sparsp_launch_count() - launches0
    clocks = sampler.finish()
    cfg.check_status()

    def avg(i):
        return sum(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(steps)) / steps

    mask_ms, dpack_ms, attn_ms = avg(0), avg(1), avg(2)
    # one step = the three calls; with an L2 flush between steps the flush itself is outside the step
    step_ms = ev[0][0].elapsed_time(end) / steps if cfg.flush is None else mask_ms + dpack_ms + attn_ms
    # demand bookkeeping alone (plan-only call), to separate the gather kernel's time
    pe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    cfg.step_plan()
    torch.cuda.synchronize()
    pe[0].record(stream)
    for _ in range(steps):
        cfg.step_plan()
    pe[1].record(stream)
    torch.cuda.synchronize()
    plan_ms = pe[0].elapsed_time(pe[1]) / steps
    return {"step": step_ms, "mask": mask_ms, "plan": plan_ms, "pack": max(dpack_ms - plan_ms, 1e-6), "attn": attn_ms,
            "launches": launches, "clocks": clocks}


def graph_replay(cfg, steps):
    """The same step captured ONCE in a CUDA graph (the three calls, nine launches) and replayed: what the launch
    gaps between the library's kernels cost.  Per-replay CUDA events; the L2 flush (small workloads) stays outside
    the timed pairs.  Returns ms per step."""
    import torch
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cfg.step()
    stream = torch.cuda.current_stream()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    cfg.check_status()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
    for s in range(steps):
        if cfg.flush is not None:
            cfg.flush.fill_(s & 0xFF)
        ev[s][0].record(stream)
        graph.replay()
        ev[s][1].record(stream)
    torch.cuda.synchronize()
    cfg.check_status()
    del graph
    return sum(e[0].elapsed_time(e[1]) for e in ev) / steps


def figures(cfg, t, peaks, traffic_table):
    """The per-kernel figures of one measured configuration."""
    attn_tflops = cfg.flops / (t["attn"] * 1e-3) / 1e12
    pack_bytes = 2.0 * cfg.volume
    pack_gbs = pack_bytes / (t["pack"] * 1e-3) / 1e9 if cfg.volume else 0.0
    traffic = traffic_table.get((cfg.wl.name, cfg.k)) if cfg.tau <= 0 and cfg.H == cfg.wl.heads else None
    return {
        "ms_per_layer": t["step"],
        "stage_ms": {"block_mask": t["mask"], "demand_plan": t["plan"], "pack": t["pack"], "sparse_attn": t["attn"]},
        "attn_tflops": attn_tflops,
        "attn_pct_bf16_peak": {"of_measured_burst": attn_tflops / peaks["bf16_tflops"],
                               "of_measured_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                               "of_nominal": attn_tflops / NOMINAL["bf16_tflops"]},
        "pack_gbs": pack_gbs,
        "pack_pct_hbm": {"of_measured": pack_gbs / peaks["hbm_gbs"], "of_nominal": pack_gbs / NOMINAL["hbm_gbs"]},
        "volume_bytes_total": cfg.volume,
        "kept_flops": cfg.flops,
        "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel (+ attn_prep_kernel, timed together)",
                     "achieved": attn_tflops, "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " burst",
                     "unit": "TFLOP/s", "frac": attn_tflops / peaks["bf16_tflops"],
                     "traffic": traffic[0] if traffic else None,
                     "traffic_source": traffic[1] if traffic else "no ncu capture of this configuration"},
        "roofline_pack": {"bound": "hbm", "kernel": "pack_bulk_kernel", "achieved": pack_gbs, "peak": peaks["hbm_gbs"],
                          "peak_source": peaks["source"], "unit": "GB/s", "frac": pack_gbs / peaks["hbm_gbs"],
                          "algorithmic_bytes": pack_bytes},
    }


def sustained_attention(cfg, seconds, local_gpu, peaks):
    """The attention call alone, back to back for `seconds`: long enough for the power cap to settle and for
    NVML's clock samples to see it; reported against the sustained tensor peak."""
    import torch
    stream = torch.cuda.current_stream()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    cfg.step_attn()
    torch.cuda.synchronize()
    e[0].record(stream)
    cfg.step_attn()
    e[1].record(stream)
    torch.cuda.synchronize()
    n = max(3, int(seconds * 1e3 / max(e[0].elapsed_time(e[1]), 1e-3)))
    sampler = ClockSampler(physical_gpu_index(local_gpu))
    sampler.start()
    e[0].record(stream)
    for _ in range(n):
        cfg.step_attn()
    e[1].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.finish()
    ms = e[0].elapsed_time(e[1]) / n
    tf = cfg.flops / (ms * 1e-3) / 1e12
    return {"calls": n, "seconds": ms * n * 1e-3, "attn_ms": ms, "attn_tflops": tf,
            "peak": peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " sustained",
            "frac": tf / peaks["bf16_tflops_sustained"], "clocks": clocks}


def end_to_end(cfg, args, barrier):
    """End to end through the public API from pinned host buffers, result read back to the host.  The path is
    independent per head, so the heads go through in a few chunks on three streams (copy in, compute, copy
    out): a chunk's kernels run while the next chunk's inputs arrive and the previous chunk's output leaves."""
    import torch
    binding, wl, dev = cfg.binding, cfg.wl, cfg.dev
    Q, K, V, O, H, P, k = cfg.Q, cfg.K, cfg.V, cfg.O, cfg.H, cfg.P, cfg.k
    stream = torch.cuda.current_stream()
    h2d = 3 * Q.numel() * 2
    d2h = O.numel() * 2 + cfg.do["volume_bytes"].numel() * 8
    hQ, hK, hV = (torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in (Q, K, V))
    hQ.copy_(Q); hK.copy_(K); hV.copy_(V)
    hO = torch.empty(O.shape, dtype=O.dtype, pin_memory=True)
    n_chunks = min(4, H) if h2d >= (32 << 20) else 1  # a small workload gains nothing from more launches
    bounds = [(c * H // n_chunks, (c + 1) * H // n_chunks) for c in range(n_chunks)]
    chunks = []
    for (h0, h1) in bounds:
        sh = binding.make_shape(h1 - h0, cfg.d, wl.grid, wl.n_text, cfg.b)
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
        binding.sparsp_demand_pack(c["shape"], c["mo"]["mask"], cfg.rank_d, P,
                                   binding.SPARSP_PLAN_ONLY if plan_only else 0,
                                   None if plan_only else K[h0:h1], None if plan_only else V[h0:h1],
                                   o["union_mask"], o["cnt"], o["seg_offset"], o["seg_total"], o["volume_bytes"],
                                   None if plan_only else c["packed"], 0 if plan_only else c["packed"].numel(),
                                   None, c["ws"])

    for c in chunks:  # size each chunk's packed buffer once (the masks are a function of the inputs)
        chunk_mask(c)
        chunk_pack(c, True)
        torch.cuda.synchronize()
        c["packed"] = torch.empty(max(int(c["do"]["seg_total"].sum().item()) * cfg.entry, 16), dtype=torch.uint8,
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
    assert int(sum(int(c["hVol"].sum().item()) for c in chunks)) == int(cfg.volume)
    return e2e_ms, n_chunks, h2d, d2h


def exchange_leg(cfg, args, rank, world):
    """The consumer-side pipeline over the transfer runtime (Export / Publish / Fetch / Release / Fence): with one
    GPU its P virtual ranks are host threads on this device, with N > 1 every process is one rank on its own GPU.
    Timed twice: pipelined (a chunk is fetched while attention runs on the previous one) and serial."""
    import torch

    from paper_2609_32197_b200 import exchange_driver
    out = {"virtual_ranks_on_one_device": world == 1, "window": args.exchange_window,
           "steady_chunks": args.exchange_chunks[0], "tail_chunks": args.exchange_chunks[1]}
    Q4, K4, V4 = cfg.Q[None], cfg.K[None], cfg.V[None]
    for mode, pipelined in (("pipelined", True), ("serial", False)):
        if world == 1:
            res = exchange_driver.run_exchange(cfg.shape, cfg.P, cfg.rank_of_block, Q4, [K4] * cfg.P, [V4] * cfg.P,
                                               cfg.mo["mask"], window=args.exchange_window,
                                               steady_chunks=args.exchange_chunks[0], tail_chunks=args.exchange_chunks[1],
                                               pipelined=pipelined, calls=3)
        else:
            res = exchange_driver.run_exchange_multi_gpu(cfg.shape, cfg.rank_of_block, Q4, K4, V4, cfg.mo["mask"],
                                                         window=args.exchange_window,
                                                         steady_chunks=args.exchange_chunks[0],
                                                         tail_chunks=args.exchange_chunks[1], pipelined=pipelined,
                                                         calls=3)
        if res.errors:
            out[mode] = {"error": "; ".join("rank %d: %s" % (r_, e) for r_, e in res.errors)}
            continue
        st = list(res.stats.values())
        out[mode] = {"ms": res.ms, "bytes_fetched_per_call": res.bytes_moved,
                     "fetches": sum(s_["fetches"] for s_ in st) // 3,
                     "acquires_that_waited": sum(s_["acquires_that_waited"] for s_ in st),
                     "ms_waiting_for_publish": sum(s_["us_waiting_for_publish"] for s_ in st) / 1e3,
                     "ms_waiting_for_release": sum(s_["us_waiting_for_release"] for s_ in st) / 1e3}
        out["slot_bytes"] = res.slot_bytes
        del res
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    import gc

    import torch
    import torch.distributed as dist

    from paper_2609_32197_b200 import binding, dist_util

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()
    peaks = load_peaks()
    traffic_table = load_attn_traffic()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl, placement = resolve_workload(args)
    pct = args.pct if args.pct else (wl.topk_pct[0] if wl.topk_pct else None)
    if args.shard == "heads" and world > 1:
        # strong scaling: ONE layer, rank r takes heads [r*H/N, (r+1)*H/N) of all three calls (every step of the
        # path is independent per head, so nothing is exchanged)
        head_range = dist_util.head_shard(wl.heads, rank, world)
        scaling = "strong"
    else:
        # weak scaling: every rank its own replica of the workload (own seed)
        wl = dist_util.replica_workload(wl, rank)
        head_range = None
        scaling = "weak"
    cfg = Config(wl, placement, pct, args.tau, dev, head_range)
    t = time_steps(cfg, args.steps, args.warmup, barrier, local)
    fig = figures(cfg, t, peaks, traffic_table)

    e2e_ms, e2e_chunks, h2d, d2h = float("nan"), 0, 3 * cfg.Q.numel() * 2, cfg.O.numel() * 2 + cfg.do["volume_bytes"].numel() * 8
    if not args.no_e2e:
        e2e_ms, e2e_chunks, h2d, d2h = end_to_end(cfg, args, barrier)
    exchange = None
    if args.exchange:
        if world > 1 and cfg.P != world:
            raise SystemExit("--exchange with N > 1 needs a workload whose rank count equals N (got %d ranks)" % cfg.P)
        exchange = exchange_leg(cfg, args, rank, world)
    sustained = None
    if world == 1 and args.sustained_s > 0:
        sustained = sustained_attention(cfg, args.sustained_s, local, peaks)

    # max over ranks (device-timed), whole-job totals
    tm, tot = dist_util.reduce_over_ranks(
        {"step": t["step"], "e2e": e2e_ms if e2e_ms == e2e_ms else 0.0},
        {"flops": cfg.flops, "launches": float(t["launches"]), "h2d": float(h2d), "d2h": float(d2h)}, dev)
    ms_per_step = tm["step"]
    if e2e_ms == e2e_ms:
        e2e_ms = tm["e2e"]
    flops_all = tot["flops"]

    result = {
        "metric": METRIC,
        "value": flops_all / (ms_per_step * 1e-3) / 1e12,
        "unit": "TFLOP/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": ms_per_step,
        "higher_is_better": True,
        "scaling": scaling,
        "vs_baseline": None,
        "dtype": "bf16",
        "data": "synthetic",
        "config": cfg.describe() | ({"sharding": "heads %d-%d of %d on rank 0" % (head_range[0], head_range[1] - 1, wl.heads)}
                                    if head_range else {}),
    }
    result.update(fig)
    result["ms_per_layer"] = ms_per_step
    result["e2e"] = {"value": None if e2e_ms != e2e_ms else flops_all / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                     "ms_per_step": None if e2e_ms != e2e_ms else e2e_ms, "head_chunks": e2e_chunks,
                     "h2d_bytes_per_step": int(tot["h2d"]), "d2h_bytes_per_step": int(tot["d2h"])}
    result["gpu_launches"] = int(tot["launches"])
    result["clocks"] = t["clocks"]
    if world == 1 and not args.no_graph:
        result["graph_ms_per_step"] = graph_replay(cfg, args.steps)
    if sustained:
        result["sustained"] = sustained
    if exchange:
        result["exchange"] = exchange
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(cfg.wl, cfg.k, placement, cfg.rank_of_block.numpy(), cfg.Q, cfg.K, cfg.V,
                                              cfg.flops, budget_s=15.0)
    if world == 1 and not args.no_per_config and args.tau <= 0 and not args.heads:
        # every configuration of the contract, measured the same way in this run (>= 10 timed iterations each)
        headline = (cfg.wl.name, cfg.k, placement)
        rows = []
        del cfg
        for (name, p_, plc) in PER_CONFIG:
            gc.collect()
            torch.cuda.empty_cache()
            from paper_2609_32197_b200 import synth
            c = Config(synth.WORKLOADS[name], plc, p_, 0.0, dev)
            tt = time_steps(c, max(10, min(args.steps, 20)), 3, barrier, local)
            row = {"config": c.describe()}
            row.update(figures(c, tt, peaks, traffic_table))
            row["clocks"] = tt["clocks"]
            row["gpu_launches"] = tt["launches"]
            if not args.no_graph:
                row["graph_ms_per_step"] = graph_replay(c, max(10, min(args.steps, 20)))
            row["is_headline_config"] = (name, c.k, plc) == headline
            rows.append(row)
            del c
        result["per_config"] = rows
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
        # every row keeps k video blocks and all text blocks: the kept pairs of the layer follow from the shape
        "config": describe_config(wl, H, k, 0.0, H * NB * (k + (NB - wl.nb_video)), placement),
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
    ap.add_argument("--workload", default="hunyuan", choices=["tiny", "mid", "cog", "wan", "hunyuan"],
                    help="headline configuration (default: the largest single-GPU one, Hunyuan-like at 10 %%)")
    ap.add_argument("--pct", type=int, default=0, help="top-k as a percentage of the video blocks")
    ap.add_argument("--tau", type=float, default=0.0, help="CDF-threshold selection with this mass instead of top-k (ours only)")
    ap.add_argument("--placement", default=None, choices=[None, "contiguous", "periodic", "shuffle"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--heads", type=int, default=0, help="override the head count (small profiling cases)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per_config list (all eight configurations)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay of the step (graph_ms_per_step)")
    ap.add_argument("--sustained-s", type=float, default=2.0,
                    help="seconds of back-to-back attention calls for the sustained figure (0 = skip)")
    ap.add_argument("--exchange", action="store_true",
                    help="also run the demand-routed exchange over the transfer runtime (pipelined vs serial)")
    ap.add_argument("--exchange-window", type=int, default=2, help="slots per rank")
    ap.add_argument("--exchange-chunks", type=int, nargs=2, default=(2, 4), help="chunks per hop: steady rounds, last round")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="with N > 1: independent replicas (weak scaling) or the heads of ONE layer split over the ranks (strong)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
