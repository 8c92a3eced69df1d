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
