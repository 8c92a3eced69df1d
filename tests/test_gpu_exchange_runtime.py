"""The transfer runtime of the demand-routed exchange (Export / Publish / Fetch / Release / Fence over a bounded
window of reusable slots) driven with virtual ranks on one device: every rank is a host thread with its own
streams; it packs per hop into a slot of its window, its consumers fetch receiver-derived byte ranges with one
asynchronous copy per planned transfer, attention runs on a chunk while the next one arrives, partial results
merge by log-sum-exp.  K and V of blocks a rank does not own are NaN in that rank's view and its receive buffer
starts out NaN, so any byte that did not travel through the exchange shows up in the result."""
import numpy as np
import pytest
import torch

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32197_b200 import binding as b
    b.lib()
    assert torch.cuda.is_available()
    return b


def _case(oracle_mod, binding, d, b, H, P, seed, k):
    from paper_2609_32197_b200 import synth
    wl = synth.Workload("xrt", H, d, (5, 11, 13), 70, b, k, None, P, seed=seed)
    Q, K, V = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    Qd, Kd = Q.cuda()[None].contiguous(), K.cuda()
    ws = binding.make_workspace(shape, P)
    ref = oracle_mod.block_mask(Q, K, b, k, wl.n_text)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, k, ws)
    assert np.array_equal(pu.u32(mo["mask"][0]), ref["mask"])
    rank = np.array([(j * 3 + j // 4) % P for j in range(NB)], np.int32)
    blk_of_tok = np.arange(N) // b
    Ks, Vs = [], []
    for r in range(P):   # rank r's view: everything it does not own is NaN
        foreign = torch.as_tensor(rank[blk_of_tok] != r)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")
        Vp[:, foreign] = float("nan")
        Ks.append(Kp.cuda()[None].contiguous())
        Vs.append(Vp.cuda()[None].contiguous())
    o_ref, lse_ref = oracle_mod.attn_all(Q, K, V, ref["mask"], b)
    return wl, shape, Qd, Ks, Vs, mo["mask"], rank, o_ref, lse_ref


def _check_result(res, P, rank, b, N, o_ref, lse_ref):
    assert not res.errors, res.errors
    for r in range(P):
        rows = np.repeat(rank == r, b)[:N]
        if not rows.any():
            continue   # a rank that owns no block (a valid degenerate placement) has no rows to check
        got = res.O[r][0].float().cpu().numpy()[:, rows]
        assert np.isfinite(got).all(), f"rank {r}: a byte that never travelled reached the result"
        err = np.abs(got - o_ref[:, rows])
        # every merge rounds the running result to bf16 once more, on top of the single-pass tolerance
        tol_max = pu.ATTN_MAX_ABS + P * 2.0 ** -9 * np.abs(o_ref[:, rows]).max()
        tol_mean = pu.ATTN_MEAN_ABS + P * 2.0 ** -10 * np.abs(o_ref[:, rows]).mean()
        assert err.max() <= tol_max and err.mean() <= tol_mean, (r, err.max(), err.mean())
        assert np.abs(res.lse[r][0].cpu().numpy()[:, rows] - lse_ref[:, rows]).max() < 2e-2


@pytest.mark.parametrize("d,b,window,steady,tail", [(128, 128, 2, 1, 2), (64, 64, 1, 2, 3), (128, 64, 3, 1, 1)])
def test_exchange_runtime_reproduces_one_shot_attention(oracle_mod, binding, d, b, window, steady, tail):
    from paper_2609_32197_b200 import exchange_driver
    H, P = 4, 4
    wl, shape, Qd, Ks, Vs, mask, rank, o_ref, lse_ref = _case(oracle_mod, binding, d, b, H, P, 81, 5 if b == 128 else 9)
    res = exchange_driver.run_exchange(shape, P, rank, Qd, Ks, Vs, mask, window=window, steady_chunks=steady,
                                       tail_chunks=tail, pipelined=True, calls=2)   # two calls: Fence and slot reuse
    _check_result(res, P, rank, b, wl.n_tokens, o_ref, lse_ref)
    for r in range(P):
        st = res.stats[r]
        # per call: one packing and one release per peer, one fetch per planned chunk; every byte of the rank's
        # exchange volume came through Fetch
        assert st["publications"] == 2 * (P - 1) and st["releases"] == 2 * (P - 1)
        assert st["fetches"] == 2 * ((P - 2) * min(steady, H) + min(tail, H))
        assert st["timeouts"] == 0
    assert sum(res.stats[r]["bytes_fetched"] for r in range(P)) == 2 * res.bytes_moved
    if window < P - 1:
        # fewer slots than hops: slots WERE reused, i.e. Release gated a later pack
        assert all(res.stats[r]["publications"] > 2 * window for r in range(P))


def test_serial_order_gives_the_same_result(oracle_mod, binding):
    from paper_2609_32197_b200 import exchange_driver
    H, P, d, b = 4, 3, 64, 128
    wl, shape, Qd, Ks, Vs, mask, rank, o_ref, lse_ref = _case(oracle_mod, binding, d, b, H, P, 83, 4)
    a = exchange_driver.run_exchange(shape, P, rank, Qd, Ks, Vs, mask, window=1, steady_chunks=2, tail_chunks=2,
                                     pipelined=False)
    c = exchange_driver.run_exchange(shape, P, rank, Qd, Ks, Vs, mask, window=2, steady_chunks=2, tail_chunks=2,
                                     pipelined=True)
    _check_result(a, P, rank, b, wl.n_tokens, o_ref, lse_ref)
    _check_result(c, P, rank, b, wl.n_tokens, o_ref, lse_ref)
    for r in range(P):   # same arithmetic in the same order: bit-identical whatever the overlap
        rows = torch.as_tensor(np.repeat(rank == r, b)[:wl.n_tokens]).cuda()
        assert torch.equal(a.O[r][0][:, rows].view(torch.int16), c.O[r][0][:, rows].view(torch.int16))


def test_pack_segment_equals_the_segment_of_the_packed_buffer(oracle_mod, binding):
    """A slot's content is exactly the (consumer, producer) run of the consumer's packed buffer as the ORACLE packs
    it; too small a slot writes nothing beyond its capacity and reports SPARSP_ERR_CAPACITY."""
    H, P, d, b = 3, 3, 64, 64
    wl, shape, Qd, Ks, Vs, mask, rank, _, _ = _case(oracle_mod, binding, d, b, H, P, 85, 7)
    from paper_2609_32197_b200 import synth
    Q, K, V = synth.make_qkv(wl, "cpu")
    Kd, Vd = K.cuda(), V.cuda()
    ws = binding.make_workspace(shape, P)
    rank_d = torch.as_tensor(rank).cuda()
    dg = pu.gpu_demand_pack(binding, shape, mask, rank_d, P, 0, Kd, Vd, ws)
    # expected bytes: the ORACLE's packed buffer, cut at the oracle's offsets
    ref = oracle_mod.block_mask(Q, K, b, 7, wl.n_text)
    dref = oracle_mod.demand(ref["mask"], rank, P, b, d)
    packed_ref = torch.as_tensor(oracle_mod.pack(K, V, dref["U"], rank, b, P, dref["total"])).cuda()
    entry = 2 * b * d * 2
    base = np.concatenate([[0], np.cumsum(dref["total"])[:-1]]) * entry
    seg, cnt = dref["seg_off"], dref["cnt"]
    assert np.array_equal(dg["cnt"][0].cpu().numpy(), cnt) and np.array_equal(dg["seg_offset"][0].cpu().numpy(), seg)
    for r in range(P):
        for p in range(P):
            if p == r:
                continue
            n = int(cnt[r, p].sum())
            lo = int(base[r]) + int(seg[r, p, 0]) * entry
            slot = torch.full((n * entry + 4096,), 0xAB, dtype=torch.uint8, device="cuda")
            # the producer's own view of K / V is enough: only blocks it owns are read
            binding.sparsp_pack_segment(shape, dg["union_mask"], rank_d, P, r, p, dg["cnt"], dg["seg_offset"], Ks[p],
                                        Vs[p], slot, n * entry, ws)
            torch.cuda.synchronize()
            assert binding.sparsp_status(ws) == binding.SPARSP_OK
            assert torch.equal(slot[:n * entry], packed_ref[lo:lo + n * entry]), (r, p)
            assert bool((slot[n * entry:] == 0xAB).all())
            if n >= 2:
                small = torch.full((n * entry,), 0xAB, dtype=torch.uint8, device="cuda")
                binding.sparsp_pack_segment(shape, dg["union_mask"], rank_d, P, r, p, dg["cnt"], dg["seg_offset"],
                                            Ks[p], Vs[p], small, (n - 1) * entry, ws)
                torch.cuda.synchronize()
                assert binding.sparsp_status(ws) == binding.SPARSP_ERR_CAPACITY
                assert torch.equal(small[:(n - 1) * entry], packed_ref[lo:lo + (n - 1) * entry])
                assert bool((small[(n - 1) * entry:] == 0xAB).all())


def test_merge_of_one_chunks_rows_matches_the_oracle_and_touches_nothing_else(oracle_mod, binding):
    """sparsp_attn_merge_rows merges only the rows of the consumer's blocks in the given heads (against the oracle's
    merge of the same rows); every other row keeps its bytes."""
    rng = np.random.default_rng(5)
    H, d, b, P = 4, 64, 64, 3
    shape = binding.make_shape(H, d, (1, 9, 37), 0, b)       # 333 tokens: 6 blocks, the last one ragged
    N, NB = 333, 6
    rank = np.array([0, 2, 1, 2, 0, 2], np.int32)
    oa = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    ob = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    la = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    lb = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    lb[0, 1, 70:80] = float("-inf")
    ro, rl = oracle_mod.attn_merge(oa.float().cpu().numpy(), la.cpu().numpy(), ob.float().cpu().numpy(), lb.cpu().numpy())
    for consumer, (h0, h1) in [(2, (1, 3)), (0, (0, 4)), (1, (3, 4))]:
        acc, acc_l = oa.clone(), la.clone()
        binding.sparsp_attn_merge_rows(shape, acc, acc_l, ob, lb, acc, acc_l, torch.as_tensor(rank).cuda(), P, consumer,
                                       h0, h1)
        torch.cuda.synchronize()
        rows = np.repeat(rank == consumer, b)[:N]
        sel = np.zeros((H, N), bool)
        sel[h0:h1, :] = rows
        got, got_l = acc[0].float().cpu().numpy(), acc_l[0].cpu().numpy()
        assert np.abs(got[sel] - ro[0][sel]).max() <= 2e-2          # bf16 rounding of the merged rows
        assert np.abs(got_l[sel] - rl[0][sel]).max() < 1e-4
        assert np.array_equal(got[~sel], oa[0].float().cpu().numpy()[~sel])   # untouched elsewhere
        assert np.array_equal(got_l[~sel], la[0].cpu().numpy()[~sel])


def test_a_consumer_that_never_fetches_times_the_producer_out(binding):
    """Host-side failure only: with a window of one slot the producer's second packing needs the first to be
    released; nobody releases it, so the bounded wait gives up with SPARSP_ERR_TIMEOUT and the endpoint lives on."""
    P, W, slot_bytes = 2, 1, 4096
    flags = torch.zeros(binding.sparsp_xchg_flag_bytes(P, W) // 4, dtype=torch.int32).pin_memory()
    slots = torch.zeros(W * slot_bytes, dtype=torch.uint8, device="cuda")
    x = binding.sparsp_xchg_export(P, 0, W, slot_bytes, slots, flags, 50_000)   # 50 ms
    binding.sparsp_xchg_fence(x)
    assert binding.sparsp_xchg_acquire(x, 0)[0] == 0
    binding.sparsp_xchg_publish(x, 0)
    torch.cuda.synchronize()
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_xchg_acquire(x, 1)
    assert e.value.code == binding.SPARSP_ERR_TIMEOUT and "release" in str(e.value)
    st = binding.sparsp_xchg_stats(x)
    assert st["timeouts"] == 1 and st["acquires_that_waited"] == 1
    # the peer releases after all (its flag store, as Release would do it): the same acquire now succeeds
    y = binding.sparsp_xchg_export(P, 1, W, slot_bytes, slots, flags, 50_000)
    binding.sparsp_xchg_fence(y)
    binding.sparsp_xchg_connect(y, 0, slots)
    dst = torch.empty(64, dtype=torch.uint8, device="cuda")
    binding.sparsp_xchg_fetch(y, 0, 0, 0, dst, 64)
    binding.sparsp_xchg_release(y, 0, 0)
    torch.cuda.synchronize()
    assert binding.sparsp_xchg_acquire(x, 1)[0] == 0
    # a fetch of something that is never published times out as well
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_xchg_fetch(y, 0, 5, 0, dst, 64)
    assert e.value.code == binding.SPARSP_ERR_TIMEOUT and "publish" in str(e.value)
    binding.sparsp_xchg_destroy(x)
    binding.sparsp_xchg_destroy(y)


def _process_rank(rank, world, port, d, b, out):
    """One PROCESS per rank (as on a node with a GPU each), both on device 0 here: slot windows are opened through
    CUDA inter-process handles, the flag page is shared host memory, the Fence's barrier a gloo barrier.  No kernel
    of one process waits for the other: every cross-rank wait is the endpoint's bounded host-side poll."""
    import os
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2609_32197_b200 import binding, exchange_driver, synth
        oracle.build()
        H, P, k = 3, world, 5 if b == 128 else 9
        wl = synth.Workload("xproc", H, d, (5, 11, 13), 70, b, k, None, P, seed=91)
        Q, K, V = synth.make_qkv(wl, "cpu")
        N, NB = wl.n_tokens, wl.n_blocks
        shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
        Qd = Q.cuda()[None].contiguous()
        ws = binding.make_workspace(shape, P)
        mo = pu.gpu_block_mask(binding, shape, Qd, K.cuda(), k, ws)
        ref = oracle.block_mask(Q, K, b, k, wl.n_text)
        assert np.array_equal(pu.u32(mo["mask"][0]), ref["mask"])
        rank_np = np.array([(j * 3 + j // 4) % P for j in range(NB)], np.int32)
        foreign = torch.as_tensor(rank_np[np.arange(N) // b] != rank)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")      # this rank's view: everything it does not own is NaN
        Vp[:, foreign] = float("nan")
        res = exchange_driver.run_exchange_multi_gpu(shape, rank_np, Qd, Kp.cuda()[None].contiguous(),
                                                     Vp.cuda()[None].contiguous(), mo["mask"], window=1,
                                                     steady_chunks=2, tail_chunks=3, calls=2, wait_limit_us=30_000_000)
        if res.errors:
            out[rank] = ("error", repr(res.errors))
            return
        o_ref, lse_ref = oracle.attn_all(Q, K, V, ref["mask"], b)
        rows = np.repeat(rank_np == rank, b)[:N]
        got = res.O[rank][0].float().cpu().numpy()[:, rows]
        err = np.abs(got - o_ref[:, rows])
        out[rank] = ("ok", bool(np.isfinite(got).all()), float(err.max()), float(err.mean()),
                     float(np.abs(o_ref[:, rows]).max()), res.stats[rank])
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("d,b", [(128, 128), (64, 64)])
def test_one_process_per_rank_through_interprocess_windows(binding, d, b):
    import socket

    import torch.multiprocessing as mp
    with socket.socket() as s_:
        s_.bind(("127.0.0.1", 0))
        port = s_.getsockname()[1]
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_process_rank, args=(world, port, d, b, out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        assert res[r][0] == "ok", res[r]
        _, finite, mx, mean, omax, st = res[r]
        assert finite, f"rank {r}: a byte that never travelled reached the result"
        assert mx <= pu.ATTN_MAX_ABS + world * 2.0 ** -9 * omax and mean <= pu.ATTN_MEAN_ABS + world * 2.0 ** -10 * omax
        assert st["publications"] == 2 and st["releases"] == 2 and st["timeouts"] == 0   # one hop per call, two calls


@pytest.mark.parametrize("case", range(16))
def test_random_exchange_configurations(oracle_mod, binding, case):
    """Shapes, rank counts (1-6, some owning nothing), random placements, windows, chunk counts, serial / pipelined and
    one or two calls drawn per case: every rank's rows equal the oracle's one-shot attention, every byte of the
    exchange volume came through Fetch, no wait ran out."""
    from paper_2609_32197_b200 import exchange_driver, synth
    rng = np.random.default_rng(4200 + case)
    while True:
        d, b = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
        H, P = int(rng.integers(1, 6)), int(rng.integers(1, 7))
        grid = (int(rng.integers(1, 6)), int(rng.integers(4, 16)), int(rng.integers(4, 20)))
        n_text = int(rng.choice([0, int(rng.integers(1, 200))]))
        wl = synth.Workload("xsweep", H, d, grid, n_text, b, 1, None, P, seed=int(rng.integers(0, 1 << 30)))
        if wl.nb_video >= 1:
            break
    N, NB = wl.n_tokens, wl.n_blocks
    k = int(rng.integers(1, wl.nb_video + 1))
    window, steady, tail = int(rng.integers(1, 4)), int(rng.integers(1, 5)), int(rng.integers(1, 5))
    pipelined, calls = bool(rng.integers(0, 2)), int(rng.integers(1, 3))
    Q, K, V = synth.make_qkv(wl, "cpu")
    shape = binding.make_shape(H, d, grid, n_text, b)
    Qd, Kd = Q.cuda()[None].contiguous(), K.cuda()
    ws = binding.make_workspace(shape, P)
    ref = oracle_mod.block_mask(Q, K, b, k, n_text)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, k, ws)
    assert np.array_equal(pu.u32(mo["mask"][0]), ref["mask"])
    rank = rng.integers(0, P, NB).astype(np.int32)
    blk_of_tok = np.arange(N) // b
    Ks, Vs = [], []
    for r in range(P):   # rank r's view: everything it does not own is NaN
        foreign = torch.as_tensor(rank[blk_of_tok] != r)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")
        Vp[:, foreign] = float("nan")
        Ks.append(Kp.cuda()[None].contiguous())
        Vs.append(Vp.cuda()[None].contiguous())
    o_ref, lse_ref = oracle_mod.attn_all(Q, K, V, ref["mask"], b)
    res = exchange_driver.run_exchange(shape, P, rank, Qd, Ks, Vs, mo["mask"], window=window, steady_chunks=steady,
                                       tail_chunks=tail, pipelined=pipelined, calls=calls, wait_limit_us=5_000_000)
    _check_result(res, P, rank, b, N, o_ref, lse_ref)
    assert sum(res.stats[r]["bytes_fetched"] for r in range(P)) == calls * res.bytes_moved
    assert all(res.stats[r]["timeouts"] == 0 for r in range(P))
