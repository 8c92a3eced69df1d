"""world_size-2 checks of the N > 1 plumbing on CPU (gloo): every rank runs its own replica, timings
reduce with MAX, work totals with SUM, and the whole-job value follows from those."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_32197_b200 import dist_util, synth
    wl = dist_util.replica_workload(synth.WORKLOADS["tiny"], rank)
    Q, _, _ = synth.make_qkv(wl, "cpu", heads=1)
    times, totals = dist_util.reduce_over_ranks({"step": 10.0 + 5 * rank, "attn": 7.0 - rank},
                                                {"flops": 1e9 * (rank + 1), "launches": 9})
    dist.barrier()
    out[rank] = (wl.seed, float(Q.float().sum()), times, totals)
    dist.destroy_process_group()


def test_two_ranks_replicas_and_reductions():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 0 and res[1][0] == 1            # each rank its own seed ...
    assert res[0][1] != res[1][1]                        # ... hence different inputs
    for r in range(world):
        times, totals = res[r][2], res[r][3]
        assert times == {"attn": 7.0, "step": 15.0}     # MAX over ranks
        assert totals == {"flops": 3e9, "launches": 18.0}  # SUM over ranks
    value = res[0][3]["flops"] / (res[0][2]["step"] * 1e-3)
    assert abs(value - 2e11) < 1


def test_single_process_passthrough():
    from paper_2609_32197_b200 import dist_util
    t, s = dist_util.reduce_over_ranks({"a": 1.5}, {"b": 2})
    assert t == {"a": 1.5} and s == {"b": 2}


def _exchange_worker(rank, world, port, out):
    """Each rank knows only the mask rows of its own query blocks (Section 5.2: it computes its demand for every
    peer, the ranks swap those, and from then on both ends of a transfer derive the same byte ranges)."""
    import numpy as np
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_32197_b200 import binding
    H, NB, b, d = 4, 24, 64, 64
    rng = np.random.default_rng(5)  # same inputs on both ranks; each then forgets the other's rows
    M = rng.random((H, NB, NB)) < 0.15
    words = np.zeros((H, NB, 1), np.uint32)
    for h, i, j in zip(*np.nonzero(M)):
        words[h, i, 0] |= np.uint32(1 << int(j))
    placement = oracle.placement_contiguous(NB, world)
    mine = words.copy()
    mine[:, placement != rank] = 0
    dem = oracle.demand(mine, placement, world, b, d)          # only row `rank` of the consumer axis is non-zero
    assert not dem["cnt"][np.arange(world) != rank].any()
    rows_c = [torch.zeros(world, H, dtype=torch.int32) for _ in range(world)]
    rows_o = [torch.zeros(world, H, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(rows_c, torch.as_tensor(dem["cnt"][rank]))
    dist.all_gather(rows_o, torch.as_tensor(dem["seg_off"][rank]))
    cnt, off = torch.stack(rows_c), torch.stack(rows_o)
    shape = binding.make_shape(H, d, (1, 1, NB * b), 0, b)
    plan = binding.sparsp_exchange_plan(shape, world, cnt[None], off[None], 2, 3)
    recs = [(t.consumer, t.producer, t.round, t.order, t.head_begin, t.head_end, t.byte_offset, t.n_bytes) for t in plan]
    full = oracle.demand(words, placement, world, b, d)
    ref = [(t["consumer"], t["producer"], t["round"], t["order"], t["head_begin"], t["head_end"], t["byte_offset"],
            t["n_bytes"]) for t in oracle.exchange_plan(full["cnt"], full["seg_off"], b, d, 2, 3)]
    out[rank] = (recs, recs == ref, int(full["volume"][rank]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_derive_the_same_transfer_list():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_exchange_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] and res[0][1] and res[1][1]   # producer's and consumer's view agree, and with the oracle
    for r in range(world):
        assert sum(t[7] for t in res[r][0] if t[0] == r) == res[r][2]   # what rank r receives is its exchange volume


def _head_shard_worker(rank, world, port, out):
    """Strong scaling by heads: rank r takes heads [r*H/N, (r+1)*H/N) of ONE layer through all three steps."""
    import numpy as np
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_32197_b200 import dist_util, synth
    wl = synth.Workload("shard", 5, 64, (3, 8, 16), 20, 64, 3, None, 3, seed=77)  # 5 heads over 2 ranks: 2 + 3
    h0, h1 = dist_util.head_shard(wl.heads, rank, world)
    Q, K, V = synth.make_qkv(wl, "cpu", heads=h1 - h0, head_begin=h0)
    placement = oracle.placement_contiguous(wl.n_blocks, wl.ranks)
    m = oracle.block_mask(Q, K, wl.block, wl.topk_abs, wl.n_text)
    dem = oracle.demand(m["mask"], placement, wl.ranks, wl.block, wl.head_dim)
    o, lse = oracle.attn_all(Q, K, V, m["mask"], wl.block)
    # the only thing that crosses ranks is the reduction of the per-rank volumes (SUM) for the report
    _, tot = dist_util.reduce_over_ranks({"step": 1.0}, {"volume": float(dem["volume"].sum())})
    out[rank] = (h0, h1, m["mask"], dem["U"], dem["cnt"], dem["volume"], o, tot["volume"])
    dist.barrier()
    dist.destroy_process_group()


def test_head_shards_concatenate_to_the_single_rank_result():
    import numpy as np

    import oracle
    from paper_2609_32197_b200 import synth
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_head_shard_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert (res[0][0], res[0][1], res[1][0], res[1][1]) == (0, 2, 2, 5)      # the shards tile the heads
    wl = synth.Workload("shard", 5, 64, (3, 8, 16), 20, 64, 3, None, 3, seed=77)
    Q, K, V = synth.make_qkv(wl, "cpu")
    placement = oracle.placement_contiguous(wl.n_blocks, wl.ranks)
    m = oracle.block_mask(Q, K, wl.block, wl.topk_abs, wl.n_text)
    dem = oracle.demand(m["mask"], placement, wl.ranks, wl.block, wl.head_dim)
    o, _ = oracle.attn_all(Q, K, V, m["mask"], wl.block)
    assert np.array_equal(np.concatenate([res[0][2], res[1][2]], axis=0), m["mask"])          # masks [H][NB][Wd]
    assert np.array_equal(np.concatenate([res[0][3], res[1][3]], axis=1), dem["U"])           # unions [P][H][Wd]
    assert np.array_equal(np.concatenate([res[0][4], res[1][4]], axis=2), dem["cnt"])         # counts [P][P][H]
    assert np.array_equal(res[0][5] + res[1][5], dem["volume"])                               # volumes add up per rank
    assert np.array_equal(np.concatenate([res[0][6], res[1][6]], axis=0), o)                  # outputs [H][N][d]
    assert res[0][7] == res[1][7] == float(dem["volume"].sum())


def _shm_addr(shm):
    import ctypes
    return ctypes.addressof(ctypes.c_char.from_buffer(shm.buf))


def _slot_protocol_worker(rank, world, port, names, out, stall_from):
    """Two processes, one exchange endpoint each, slots and flag page in inter-process shared memory (host-memory
    endpoints: copies are memcpy, so the protocol runs without a GPU).  Each rank packs `n_uses` payloads for its peer
    into a window of 2 slots and consumes the peer's; rank 1 sleeps before every fetch, so rank 0, which does not,
    must wait for Release before it re-packs a slot (and would overwrite an unread slot if it did not).  With `stall_from` >= 0 rank 1 stops
    releasing from that use on: rank 0's bounded wait for the slot must end in SPARSP_ERR_TIMEOUT."""
    import time
    from multiprocessing import shared_memory

    import numpy as np
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_32197_b200 import binding as b
    W, slot_bytes, n_uses = 2, 1 << 16, 6
    shm_flags = shared_memory.SharedMemory(name=names["flags"])
    shm_slots = [shared_memory.SharedMemory(name=names["slots%d" % r]) for r in range(world)]
    x = b.sparsp_xchg_export(world, rank, W, slot_bytes, _shm_addr(shm_slots[rank]), _shm_addr(shm_flags), 300_000,
                             b.SPARSP_XCHG_HOST_MEMORY)
    peer = 1 - rank
    b.sparsp_xchg_connect(x, peer, _shm_addr(shm_slots[peer]))
    dist.barrier()            # Fence: the barrier across ranks, then the next epoch
    b.sparsp_xchg_fence(x)
    mine = np.ndarray((W, slot_bytes), np.uint8, buffer=shm_slots[rank].buf)
    recv = np.zeros(slot_bytes, np.uint8)
    import ctypes
    log = {"acquired": [], "bad_payload": 0, "timeout": None, "consumed": 0}

    def produce(u):
        slot, _ = b.sparsp_xchg_acquire(x, u)
        mine[slot, :] = (17 * rank + u) % 251      # the "pack"
        b.sparsp_xchg_publish(x, u, 0)
        log["acquired"].append((u, slot))

    def consume(u):
        if rank == 1:
            time.sleep(0.03)                        # a slow consumer
        b.sparsp_xchg_fetch(x, peer, u, 0, recv.ctypes.data, slot_bytes, 0)
        if not (recv == (17 * peer + u) % 251).all():
            log["bad_payload"] += 1
        log["consumed"] += 1
        if not (rank == 1 and 0 <= stall_from <= u):
            b.sparsp_xchg_release(x, peer, u, 0)

    try:
        for u in range(min(W, n_uses)):
            produce(u)
        for u in range(n_uses):
            consume(u)
            if u + W < n_uses:
                produce(u + W)
    except b.SparspError as exc:
        log["timeout"] = (exc.code, str(exc))
    log["stats"] = b.sparsp_xchg_stats(x)
    out[rank] = log
    b.sparsp_xchg_destroy(x)
    del mine
    for s_ in [shm_flags] + shm_slots:
        s_.close()
    try:
        dist.barrier()
    except Exception:  # noqa: BLE001  (the peer may have left after its timeout)
        pass
    dist.destroy_process_group()


def _run_slot_protocol(stall_from):
    from multiprocessing import shared_memory

    from paper_2609_32197_b200 import binding as b
    world, W, slot_bytes = 2, 2, 1 << 16
    shms = {"flags": shared_memory.SharedMemory(create=True, size=max(b.sparsp_xchg_flag_bytes(world, W), 64))}
    for r in range(world):
        shms["slots%d" % r] = shared_memory.SharedMemory(create=True, size=W * slot_bytes)
    for s_ in shms.values():
        s_.buf[:] = bytes(len(s_.buf))
    try:
        with mp.Manager() as mgr:
            out = mgr.dict()
            names = {k: v.name for k, v in shms.items()}
            mp.spawn(_slot_protocol_worker, args=(world, _free_port(), names, out, stall_from), nprocs=world, join=True)
            return dict(out)
    finally:
        for s_ in shms.values():
            s_.close()
            s_.unlink()


def test_slot_window_protocol_between_two_processes():
    res = _run_slot_protocol(stall_from=-1)
    for r in (0, 1):
        log = res[r]
        assert log["timeout"] is None and log["bad_payload"] == 0 and log["consumed"] == 6
        assert log["acquired"] == [(u, u % 2) for u in range(6)]            # six payloads through two slots
        st = log["stats"]
        assert st["publications"] == 6 and st["fetches"] == 6 and st["releases"] == 6 and st["timeouts"] == 0
        assert st["bytes_fetched"] == 6 * (1 << 16)
    assert res[0]["stats"]["acquires_that_waited"] >= 1                      # Release did gate the fast rank's later packs


def test_a_consumer_that_stops_releasing_times_the_producer_out():
    res = _run_slot_protocol(stall_from=1)
    from paper_2609_32197_b200 import binding as b
    # rank 1 consumed everything rank 0 could publish (uses 0..2: slot 1 is never returned after use 1, so use 3
    # cannot be packed) and saw only intact payloads; rank 0's wait for the slot of use 3 ran out
    assert res[0]["timeout"] is not None and res[0]["timeout"][0] == b.SPARSP_ERR_TIMEOUT
    assert "release" in res[0]["timeout"][1]
    assert [u for u, _ in res[0]["acquired"]] == [0, 1, 2]
    assert res[0]["stats"]["timeouts"] == 1
    assert res[0]["bad_payload"] == 0 and res[1]["bad_payload"] == 0
    # rank 1 in turn loses its consumer (rank 0 has left before reading use 2): the slot of its use 4 is never
    # returned and its own bounded wait gives up as well
    assert res[1]["timeout"] is not None and res[1]["timeout"][0] == b.SPARSP_ERR_TIMEOUT
    assert "release" in res[1]["timeout"][1] and res[1]["consumed"] == 3
    assert [u for u, _ in res[1]["acquired"]] == [0, 1, 2, 3]
