"""Drives the demand-routed exchange (Sections 5-7) with P virtual ranks on ONE device.

Every virtual rank is a host thread with its own streams (pack, copy, compute), workspaces, slot window, receive
buffer and running attention result -- what a process per GPU would own on a node.  The ranks meet only through
the exchange endpoints (sparsp_xchg_*): slot windows that peers address directly and the shared flag page.  No
kernel waits for another rank; a rank's host thread waits (bounded) for a publication before it enqueues a copy
and for a release before it re-packs a slot.

Per attention call and rank r (the plan comes from sparsp_exchange_plan, the same list on every rank):
    Fence (barrier across ranks, next epoch)
    attention over r's own blocks                                     -> running result
    producer side, up to `window` packings ahead:
        Acquire slot (k mod window) -> pack what rank (r + k + 1) mod P selected from r -> Publish
    for round k = 0 .. P-2, producer p = (r - (k + 1)) mod P, chunk by chunk in the plan's order:
        Fetch the chunk's byte range from p's slot into r's receive buffer (copy stream, copy engines)
        Release p's slot after the hop's last chunk
        compute stream: wait for the copy -> attention on the chunk's heads, remote tiles read in place from the
        receive buffer -> log-sum-exp merge into the running result
        (the copy stream is already fetching the next chunk meanwhile; with pipelined=False it waits for the
        attention of the previous chunk instead, which gives the serial time to compare with)
This module only orders library calls; every step runs in the library's kernels or on the copy engines.
"""
from __future__ import annotations

import threading
import time

import torch

from . import binding


class ExchangeResult:
    def __init__(self):
        self.O = {}          # rank -> [1][H][N][d] bf16 (rows of the rank's own query blocks are meaningful)
        self.lse = {}        # rank -> [1][H][N] fp32
        self.stats = {}      # rank -> dict of endpoint counters
        self.errors = []     # (rank, exception)
        self.ms = None       # device time of the whole call (max over ranks), if timed
        self.slot_bytes = 0
        self.bytes_moved = 0


def _rank_thread(r, ctx, res, barrier):
    """One rank's attention call(s): a host thread of a virtual rank, or the only thread of a process that owns
    a GPU.  `barrier` is the Fence's barrier across ranks (wait() / abort())."""
    b_ = binding
    P, W, shape = ctx["P"], ctx["window"], ctx["shape"]
    dev = ctx["dev"]
    try:
        torch.cuda.set_device(dev)
        s_pack, s_copy, s_comp = (torch.cuda.Stream(dev) for _ in range(3))
        x = b_.sparsp_xchg_export(P, r, W, ctx["slot_bytes"], ctx["slots"][r], ctx["flag_page"], ctx["wait_limit_us"])
        for p in range(P):
            if p != r:
                b_.sparsp_xchg_connect(x, p, ctx["slots"][p])
        Q, K, V = ctx["Q"], ctx["K"][r], ctx["V"][r]
        H, N = shape.heads, ctx["N"]
        mask, rank_d = ctx["mask"], ctx["rank_d"]
        U, cnt, seg_off, seg_total = ctx["U"], ctx["cnt"], ctx["seg_off"], ctx["seg_total"]
        entry = ctx["entry"]
        ws_pack, ws_attn = ctx["ws_pack"][r], ctx["ws_attn"][r]
        recv = ctx["recv"][r]
        base_d = ctx["recv_base"][r]
        plan = ctx["plan"][r]
        seg_first = ctx["seg_first"]      # host: first entry of (consumer, producer) inside the consumer's buffer
        with torch.cuda.stream(s_comp):
            acc = torch.zeros_like(Q)
            acc_lse = torch.full((1, H, N), float("-inf"), dtype=torch.float32, device=dev)
            part = torch.zeros_like(Q)
            part_lse = torch.full((1, H, N), float("-inf"), dtype=torch.float32, device=dev)
            hop = torch.empty_like(mask)
        for st in (s_pack, s_copy, s_comp):
            st.synchronize()
        n_calls = ctx["calls"]
        t_ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for call in range(n_calls):
            timed = call == n_calls - 1
            # ---- Fence: everybody's copies of the previous call are complete, then the next epoch
            s_copy.synchronize()
            s_comp.synchronize()
            barrier.wait()
            b_.sparsp_xchg_fence(x)
            if timed:
                t_ev[0].record(s_comp)

            def produce(u):
                c = (r + u + 1) % P
                _, ptr = b_.sparsp_xchg_acquire(x, u)
                with torch.cuda.stream(s_pack):
                    b_.sparsp_pack_segment(shape, U, rank_d, P, c, r, cnt, seg_off, K, V, ptr, ctx["slot_bytes"], ws_pack)
                b_.sparsp_xchg_publish(x, u, s_pack)

            # ---- local blocks first: no communication
            with torch.cuda.stream(s_comp):
                b_.sparsp_hop_mask(shape, mask, rank_d, P, r, r, hop)
                b_.sparsp_sparse_attn_fwd(shape, Q, K, V, hop, 0.0, acc, acc_lse, ws_attn)
            for u in range(min(W, P - 1)):
                produce(u)
            for k in range(P - 1):
                p = (r - (k + 1)) % P
                chunks = plan[k]
                hop_start = seg_first[r][p] * entry
                for ci, t in enumerate(chunks):
                    if not ctx["pipelined"]:
                        s_copy.wait_stream(s_comp)   # serial: no copy while attention runs
                    b_.sparsp_xchg_fetch(x, p, k, t.byte_offset - hop_start, recv.data_ptr() + t.byte_offset, t.n_bytes,
                                         s_copy)
                    arrived = torch.cuda.Event()
                    arrived.record(s_copy)
                    if ci == len(chunks) - 1:
                        b_.sparsp_xchg_release(x, p, k, s_copy)
                    if t.n_entries == 0:
                        continue
                    with torch.cuda.stream(s_comp):
                        s_comp.wait_event(arrived)
                        b_.sparsp_hop_chunk_mask(shape, mask, rank_d, P, r, p, t.head_begin, t.head_end, hop)
                        b_.sparsp_sparse_attn_fwd_packed(shape, Q, K, V, hop, rank_d, P, r, U, seg_off, seg_total, recv,
                                                         ctx["recv_capacity"][r], base_d, 0.0, part, part_lse, ws_attn)
                        b_.sparsp_attn_merge_rows(shape, acc, acc_lse, part, part_lse, acc, acc_lse, rank_d, P, r,
                                                  t.head_begin, t.head_end)
                if k + W < P - 1:
                    produce(k + W)
            if timed:
                s_comp.wait_stream(s_copy)
                s_comp.wait_stream(s_pack)
                t_ev[1].record(s_comp)
        for st in (s_pack, s_copy, s_comp):
            st.synchronize()
        for ws in (ws_pack, ws_attn):
            code = b_.sparsp_status(ws)
            if code != b_.SPARSP_OK:
                raise b_.SparspError(code, b_.sparsp_last_error())
        res.O[r], res.lse[r] = acc, acc_lse
        res.stats[r] = b_.sparsp_xchg_stats(x)
        res.stats[r]["ms"] = t_ev[0].elapsed_time(t_ev[1])
        b_.sparsp_xchg_destroy(x)
    except Exception as exc:  # noqa: BLE001  (reported to the caller, which decides)
        res.errors.append((r, exc))
        try:
            barrier.abort()
        except Exception:  # noqa: BLE001
            pass


def run_exchange(shape, n_ranks, rank_of_block, Q, K_of_rank, V_of_rank, mask, window=2, steady_chunks=1,
                 tail_chunks=1, pipelined=True, calls=1, wait_limit_us=20_000_000, device=None):
    """One (or `calls` successive) attention call(s) over the demand-routed exchange with `n_ranks` virtual ranks.

    Q [1][H][N][d] and mask are shared (a rank only ever computes the rows of its own query blocks); K_of_rank[r] /
    V_of_rank[r] are rank r's view of K and V -- only the blocks r owns are ever read from them.  Returns an
    ExchangeResult; rows of rank r's query blocks in result.O[r] are the attention output."""
    b_ = binding
    dev = torch.device(device if device is not None else Q.device)
    P = n_ranks
    g = b_.sparsp_geometry(shape)
    entry = 2 * shape.block * shape.head_dim * 2
    rank_d = torch.as_tensor(rank_of_block, dtype=torch.int32).to(dev)
    # the complete communication plan, established once per attention call (Section 5.2)
    do = b_.alloc_demand_outputs(shape, P, dev)
    ws0 = b_.make_workspace(shape, P, dev)
    b_.sparsp_demand_pack(shape, mask, rank_d, P, b_.SPARSP_PLAN_ONLY, None, None, do["union_mask"], do["cnt"],
                          do["seg_offset"], do["seg_total"], do["volume_bytes"], None, 0, None, ws0)
    torch.cuda.synchronize(dev)
    cnt_h = do["cnt"][0].cpu()
    seg_h = do["seg_offset"][0].cpu()
    tot_h = do["seg_total"][0].cpu()
    transfers = b_.sparsp_exchange_plan(shape, P, do["cnt"], do["seg_offset"], steady_chunks, tail_chunks)
    plan = {r: {k: [] for k in range(P - 1)} for r in range(P)}
    for t in transfers:
        plan[t.consumer][t.round].append(t)
    for r in range(P):
        for k in range(P - 1):
            plan[r][k].sort(key=lambda t: t.order)
    # same slot geometry on every rank: the largest (consumer, producer) payload (Section 6.2)
    pair_entries = cnt_h.sum(dim=2)
    slot_bytes = max(int(pair_entries[r, p]) for r in range(P) for p in range(P) if p != r) * entry if P > 1 else entry
    slot_bytes = max(slot_bytes, entry)
    res = ExchangeResult()
    res.slot_bytes = slot_bytes
    res.bytes_moved = int(do["volume_bytes"].sum().item())
    flag_page = torch.zeros(b_.sparsp_xchg_flag_bytes(P, window) // 4, dtype=torch.int32).pin_memory()
    ctx = dict(P=P, window=window, shape=shape, dev=dev, slot_bytes=slot_bytes, flag_page=flag_page,
               wait_limit_us=wait_limit_us, Q=Q, K=K_of_rank, V=V_of_rank, N=g.n_tokens, mask=mask, rank_d=rank_d,
               U=do["union_mask"], cnt=do["cnt"], seg_off=do["seg_offset"], seg_total=do["seg_total"], entry=entry,
               plan=plan, pipelined=pipelined, calls=calls,
               seg_first=[[int(seg_h[r, p, 0]) for p in range(P)] for r in range(P)],
               slots=[torch.empty(window * slot_bytes, dtype=torch.uint8, device=dev) for _ in range(P)],
               ws_pack=[b_.make_workspace(shape, P, dev) for _ in range(P)],
               ws_attn=[b_.make_workspace(shape, P, dev) for _ in range(P)],
               # a rank's receive buffer: its packed buffer, NaN until a Fetch fills a range (0xFFFF is a bf16 NaN)
               recv=[torch.full((max(int(tot_h[r]) * entry, entry) + 64,), 0xFF, dtype=torch.uint8, device=dev)
                     for r in range(P)],
               recv_capacity=[max(int(tot_h[r]) * entry, entry) for r in range(P)],
               recv_base=[torch.zeros(1, P, dtype=torch.int64, device=dev) for _ in range(P)])
    torch.cuda.synchronize(dev)
    barrier = threading.Barrier(P)
    threads = [threading.Thread(target=_rank_thread, args=(r, ctx, res, barrier), daemon=True) for r in range(P)]
    t0 = time.perf_counter()
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    res.wall_s = time.perf_counter() - t0
    if not res.errors:
        res.ms = max(res.stats[r]["ms"] for r in range(P))
    return res


class _DistBarrier:
    """The Fence's barrier across processes (one rank per GPU)."""

    def wait(self):
        import torch.distributed as dist
        dist.barrier()

    def abort(self):
        pass


def run_exchange_multi_gpu(shape, rank_of_block, Q, K, V, mask, window=2, steady_chunks=1, tail_chunks=1,
                           pipelined=True, calls=1, wait_limit_us=20_000_000):
    """The same attention call with ONE RANK PER PROCESS AND GPU (torch.distributed initialised; rank = GPU).
    Every rank holds Q, mask and its view of K / V on its own device (only the blocks it owns are read), computes
    the demand plan locally (the masks are identical on all ranks), exports a slot window in its own memory and
    opens its peers' windows through CUDA inter-process handles; the flag page is inter-process shared host
    memory created by rank 0.  Fetch is then a peer copy over NVLink into the consumer's own memory; every wait is
    the endpoint's bounded host-side poll.  Returns this rank's ExchangeResult."""
    import torch.distributed as dist
    from multiprocessing import shared_memory
    from torch.multiprocessing.reductions import reduce_tensor
    b_ = binding
    r, P = dist.get_rank(), dist.get_world_size()
    dev = Q.device
    g = b_.sparsp_geometry(shape)
    entry = 2 * shape.block * shape.head_dim * 2
    rank_d = torch.as_tensor(rank_of_block, dtype=torch.int32).to(dev)
    do = b_.alloc_demand_outputs(shape, P, dev)
    ws0 = b_.make_workspace(shape, P, dev)
    b_.sparsp_demand_pack(shape, mask, rank_d, P, b_.SPARSP_PLAN_ONLY, None, None, do["union_mask"], do["cnt"],
                          do["seg_offset"], do["seg_total"], do["volume_bytes"], None, 0, None, ws0)
    torch.cuda.synchronize(dev)
    cnt_h, seg_h, tot_h = do["cnt"][0].cpu(), do["seg_offset"][0].cpu(), do["seg_total"][0].cpu()
    transfers = b_.sparsp_exchange_plan(shape, P, do["cnt"], do["seg_offset"], steady_chunks, tail_chunks)
    plan = {r: {k: [] for k in range(P - 1)}}
    for t in transfers:
        if t.consumer == r:
            plan[r][t.round].append(t)
    for k in range(P - 1):
        plan[r][k].sort(key=lambda t: t.order)
    pair_entries = cnt_h.sum(dim=2)
    slot_bytes = max([int(pair_entries[c, p]) for c in range(P) for p in range(P) if p != c] + [1]) * entry
    # Export: this rank's window, opened by every peer through an inter-process handle
    my_slots = torch.empty(window * slot_bytes, dtype=torch.uint8, device=dev)
    rebuild, args = reduce_tensor(my_slots)
    gathered = [None] * P
    dist.all_gather_object(gathered, args)
    slots = {p: (my_slots if p == r else rebuild(*gathered[p])) for p in range(P)}
    # flag page: shared host memory, created and zero-filled by rank 0
    n_flag = b_.sparsp_xchg_flag_bytes(P, window)
    name = [None]
    shm = None
    if r == 0:
        shm = shared_memory.SharedMemory(create=True, size=max(n_flag, 64))
        shm.buf[:] = bytes(len(shm.buf))
        name[0] = shm.name
    dist.broadcast_object_list(name, src=0)
    if r != 0:
        shm = shared_memory.SharedMemory(name=name[0])
    import ctypes
    flag_addr = ctypes.addressof(ctypes.c_char.from_buffer(shm.buf))
    res = ExchangeResult()
    res.slot_bytes = slot_bytes
    res.bytes_moved = int(do["volume_bytes"].sum().item())
    cap = max(int(tot_h[r]) * entry, entry)
    ctx = dict(P=P, window=window, shape=shape, dev=dev, slot_bytes=slot_bytes, flag_page=flag_addr,
               wait_limit_us=wait_limit_us, Q=Q, K={r: K}, V={r: V}, N=g.n_tokens, mask=mask, rank_d=rank_d,
               U=do["union_mask"], cnt=do["cnt"], seg_off=do["seg_offset"], seg_total=do["seg_total"], entry=entry,
               plan=plan, pipelined=pipelined, calls=calls,
               seg_first=[[int(seg_h[c, p, 0]) for p in range(P)] for c in range(P)], slots=slots,
               ws_pack={r: b_.make_workspace(shape, P, dev)}, ws_attn={r: b_.make_workspace(shape, P, dev)},
               recv={r: torch.full((cap + 64,), 0xFF, dtype=torch.uint8, device=dev)}, recv_capacity={r: cap},
               recv_base={r: torch.zeros(1, P, dtype=torch.int64, device=dev)})
    torch.cuda.synchronize(dev)
    dist.barrier()
    _rank_thread(r, ctx, res, _DistBarrier())
    dist.barrier()
    del slots
    shm.close()
    if r == 0:
        shm.unlink()
    if not res.errors:
        res.ms = res.stats[r]["ms"]
    return res
