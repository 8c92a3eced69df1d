"""Consumer-side pipeline on the GPU: per-hop masks, per-hop partial attention with log-sum-exp
output, and the merge of the partial results -- against the oracle's versions of the same steps and
against attention over all kept blocks at once."""
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


@pytest.mark.parametrize("d,b,layout", [(128, 128, "HND"), (64, 64, "NHD"), (128, 64, "HND")])
def test_hop_partials_merge_to_full_attention(oracle_mod, binding, d, b, layout):
    from paper_2609_32197_b200 import synth
    H, P = 3, 3
    wl = synth.Workload("hop", H, d, (5, 11, 13), 70, b, 3 if b == 128 else 5, None, P, seed=51)
    Q, K, V = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    Qd, Kd, Vd = (pu.to_layout(x.cuda(), layout) for x in (Q, K, V))
    ws = binding.make_workspace(shape, P)
    ref = oracle_mod.block_mask(Q, K, b, wl.topk_abs, wl.n_text)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.topk_abs, ws)
    rank = np.array([(j * 2) % P for j in range(NB)], np.int32)
    rank_d = torch.as_tensor(rank).cuda()

    # attention over everything at once (reference for the merged result)
    O_full = torch.zeros_like(Qd)
    lse_full = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mo["mask"], 0.0, O_full, lse_full, ws)
    o_ref, lse_ref = oracle_mod.attn_all(Q, K, V, ref["mask"], b)

    hop = torch.empty_like(mo["mask"])
    for r in range(P):
        acc = torch.zeros_like(Qd)
        acc_lse = torch.full((1, H, N), float("-inf"), dtype=torch.float32, device="cuda")
        for p in range(P):
            binding.sparsp_hop_mask(shape, mo["mask"], rank_d, P, r, p, hop)
            assert np.array_equal(pu.u32(hop[0]), oracle_mod.hop_mask(ref["mask"], rank, r, p)), (r, p)
            part = torch.zeros_like(Qd)
            part_lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
            binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, hop, 0.0, part, part_lse, ws)
            binding.sparsp_attn_merge(shape, acc, acc_lse, part, part_lse, acc, acc_lse)  # in place
        torch.cuda.synchronize()
        assert binding.sparsp_status(ws) == binding.SPARSP_OK
        rows = np.repeat(rank == r, b)[:N]
        got = pu.from_layout(acc, layout).float().cpu().numpy()[:, rows]
        err = np.abs(got - o_ref[:, rows])
        # every merge rounds the running result to bf16 once more (half an ulp = 2^-9 relative), on
        # top of the single-pass attention tolerance
        tol_max = pu.ATTN_MAX_ABS + P * 2.0 ** -9 * np.abs(o_ref[:, rows]).max()
        tol_mean = pu.ATTN_MEAN_ABS + P * 2.0 ** -10 * np.abs(o_ref[:, rows]).mean()
        assert err.max() <= tol_max and err.mean() <= tol_mean, (r, err.max(), err.mean(), tol_max, tol_mean)
        assert np.abs(acc_lse[0].cpu().numpy()[:, rows] - lse_ref[:, rows]).max() < 2e-2
        # and against the one-shot kernel result (two bf16 roundings apart at most)
        one = pu.from_layout(O_full, layout).float().cpu().numpy()[:, rows]
        assert np.abs(got - one).max() <= tol_max
        # rows of other ranks: nothing arrived -> zeros, lse = -inf
        assert not pu.from_layout(acc, layout).float().cpu().numpy()[:, ~rows].any()
        assert np.all(np.isneginf(acc_lse[0].cpu().numpy()[:, ~rows]))


def test_merge_kernel_matches_oracle_elementwise(oracle_mod, binding):
    rng = np.random.default_rng(3)
    H, N, d = 2, 300, 64
    shape = binding.make_shape(H, d, (1, 10, 30), 0, 64)
    oa = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    ob = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    la = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    lb = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    la[0, 0, :5] = float("-inf")
    lb[0, 1, :5] = float("-inf")
    la[0, 1, 7] = lb[0, 1, 7] = float("-inf")
    out = torch.empty_like(oa)
    lse = torch.empty_like(la)
    binding.sparsp_attn_merge(shape, oa, la, ob, lb, out, lse)
    torch.cuda.synchronize()
    ro, rl = oracle_mod.attn_merge(oa.float().cpu().numpy(), la.cpu().numpy(), ob.float().cpu().numpy(), lb.cpu().numpy())
    assert np.abs(out.float().cpu().numpy() - ro).max() <= 2e-2  # bf16 output rounding
    fin = np.isfinite(rl)
    assert np.abs(lse.cpu().numpy()[fin] - rl[fin]).max() < 1e-4
    assert np.array_equal(np.isneginf(lse.cpu().numpy()), np.isneginf(rl))


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("alias", ["a", "b"])
def test_merge_in_place_equals_out_of_place(binding, d, alias):
    """O / lse may alias either input: the result must be bit for bit the out-of-place one."""
    rng = np.random.default_rng(9 + d)
    H, N = 3, 333
    shape = binding.make_shape(H, d, (1, 9, 37), 0, 64)
    oa = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    ob = torch.tensor(rng.standard_normal((1, H, N, d)), dtype=torch.float32).to(torch.bfloat16).cuda()
    la = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    lb = torch.tensor(rng.standard_normal((1, H, N)) * 3, dtype=torch.float32).cuda()
    la[0, 0, :7] = float("-inf")
    lb[0, 0, 3:11] = float("-inf")
    out, lse = torch.empty_like(oa), torch.empty_like(la)
    binding.sparsp_attn_merge(shape, oa, la, ob, lb, out, lse)
    xa, xla, xb, xlb = oa.clone(), la.clone(), ob.clone(), lb.clone()
    if alias == "a":
        binding.sparsp_attn_merge(shape, xa, xla, xb, xlb, xa, xla)
        got, got_l = xa, xla
    else:
        binding.sparsp_attn_merge(shape, xa, xla, xb, xlb, xb, xlb)
        got, got_l = xb, xlb
    torch.cuda.synchronize()
    assert torch.equal(got.view(torch.int16), out.view(torch.int16))
    assert torch.equal(got_l.view(torch.int32), lse.view(torch.int32))


@pytest.mark.parametrize("d,b,layout", [(128, 128, "HND"), (64, 64, "HND"), (128, 64, "NHD"), (64, 128, "HND")])
@pytest.mark.parametrize("v_scale", [1.0, 0.5])
def test_attention_reading_remote_blocks_from_the_packed_buffer(oracle_mod, binding, d, b, layout, v_scale):
    """The consumer-side attention must produce the consumer's rows from its own K/V blocks plus its
    packed buffer alone: the K/V handed to it have every block the consumer does NOT own overwritten
    with NaN, and the oracle computes the expected rows from the same restricted view."""
    from paper_2609_32197_b200 import synth
    H, P = 3, 3
    wl = synth.Workload("packed", H, d, (5, 11, 13), 70, b, 5 if b == 128 else 9, None, P, seed=61)
    Q, K, V = synth.make_qkv(wl, "cpu")
    V = (V.float() * v_scale).to(torch.bfloat16)  # 1: the generator's own V ~ N(0,1); 0.5: an extra case
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    Qd, Kd, Vd = (pu.to_layout(x.cuda(), layout) for x in (Q, K, V))
    ws = binding.make_workspace(shape, P)
    ref = oracle_mod.block_mask(Q, K, b, wl.topk_abs, wl.n_text)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.topk_abs, ws)
    rank = np.array([(j * 2 + j // 3) % P for j in range(NB)], np.int32)
    rank_d = torch.as_tensor(rank).cuda()
    dg = pu.gpu_demand_pack(binding, shape, mo["mask"], rank_d, P, 0, Kd, Vd, ws)
    dref = oracle_mod.demand(ref["mask"], rank, P, b, d)
    packed_ref = oracle_mod.pack(K, V, dref["U"], rank, b, P, dref["total"])
    assert np.array_equal(dg["packed"].cpu().numpy()[:packed_ref.size], packed_ref)
    blk_of_tok = np.arange(N) // b
    for r in range(P):
        # poison everything the consumer does not own
        foreign = torch.as_tensor(rank[blk_of_tok] != r)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")
        Vp[:, foreign] = float("nan")
        Kpd, Vpd = pu.to_layout(Kp.cuda(), layout), pu.to_layout(Vp.cuda(), layout)
        O = torch.full_like(Qd, 7.0)
        lse = torch.full((1, H, N), 7.0, dtype=torch.float32, device="cuda")
        binding.sparsp_sparse_attn_fwd_packed(shape, Qd, Kpd, Vpd, mo["mask"], rank_d, P, r, dg["union_mask"],
                                              dg["seg_offset"], dg["seg_total"], dg["packed"],
                                              dg["packed"].numel() - 64, None, 0.0, O, lse, ws)
        torch.cuda.synchronize()
        assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
        # oracle: attention over the consumer's restricted view (NaN outside local + packed blocks)
        Kr, Vr = oracle_mod.consumer_view(K, V, packed_ref, dref, rank, b, r)
        units = [(h, i) for h in range(H) for i in range(NB) if rank[i] == r]
        Kv = torch.tensor(Kr[:, :N]).to(torch.bfloat16)
        Vv = torch.tensor(Vr[:, :N]).to(torch.bfloat16)
        got = pu.from_layout(O, layout)
        mx, mean = pu.check_attn_units(oracle_mod, Q, Kv, Vv, ref["mask"], b, got, units, lse_gpu=lse[0])
        # rows of other ranks are left as they were
        other = torch.as_tensor(np.repeat(rank != r, b)[:N])
        assert bool((got[:, other].float() == 7.0).all()) and bool((lse[0][:, other] == 7.0).all())


def test_packed_attention_with_explicit_slot_bases(oracle_mod, binding):
    """Consumer slots placed out of order with a gap between them: the attention finds its tiles
    through the same bases the pack call was given."""
    from paper_2609_32197_b200 import synth
    H, P, d, b = 2, 2, 64, 64
    wl = synth.Workload("packed_base", H, d, (4, 9, 11), 40, b, 6, None, P, seed=62)
    Q, K, V = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    Qd, Kd, Vd = (x.cuda() for x in (Q, K, V))
    ws = binding.make_workspace(shape, P)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.topk_abs, ws)
    rank = (np.arange(NB) % P).astype(np.int32)
    rank_d = torch.as_tensor(rank).cuda()
    plan = pu.gpu_demand_pack(binding, shape, mo["mask"], rank_d, P, binding.SPARSP_PLAN_ONLY, None, None, ws)
    tot = plan["seg_total"][0].cpu().numpy()
    entry = 2 * b * d * 2
    base = np.array([[(int(tot[1]) + 3) * entry, 0]], np.int64)      # rank 1 first, 3 entries of gap, then rank 0
    base_d = torch.as_tensor(base).cuda()
    cap = int(tot.sum()) + 3
    dg = pu.gpu_demand_pack(binding, shape, mo["mask"], rank_d, P, 0, Kd, Vd, ws, capacity_entries=cap, dst_base=base_d)
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    mask_np = pu.u32(mo["mask"][0])
    blk_of_tok = np.arange(N) // b
    for r in range(P):
        foreign = torch.as_tensor(rank[blk_of_tok] != r)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")
        Vp[:, foreign] = float("nan")
        O = torch.zeros_like(Qd)
        lse = torch.zeros((1, H, N), dtype=torch.float32, device="cuda")
        binding.sparsp_sparse_attn_fwd_packed(shape, Qd, Kp.cuda(), Vp.cuda(), mo["mask"], rank_d, P, r,
                                              dg["union_mask"], dg["seg_offset"], dg["seg_total"], dg["packed"],
                                              cap * entry, base_d, 0.0, O, lse, ws)
        torch.cuda.synchronize()
        assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
        units = [(h, i) for h in range(H) for i in range(NB) if rank[i] == r]
        pu.check_attn_units(oracle_mod, Q, K, V, mask_np, b, O, units, lse_gpu=lse[0])


def test_packed_attention_rejects_bad_arguments(binding):
    shape = binding.make_shape(2, 64, (2, 4, 8), 0, 64)
    ws = binding.make_workspace(shape, 2)
    z = torch.zeros(64, dtype=torch.uint8, device="cuda")
    for consumer, cap in [(2, 1 << 20), (-1, 1 << 20), (0, -5)]:
        with pytest.raises(RuntimeError):
            binding.sparsp_sparse_attn_fwd_packed(shape, z, z, z, z, z, 2, consumer, z, z, z, z, cap, None, 0.0, z,
                                                  None, ws)


@pytest.mark.parametrize("d,b,steady,tail", [(128, 128, 1, 1), (64, 64, 2, 3), (128, 64, 3, 2)])
@pytest.mark.parametrize("v_scale", [1.0, 0.5])
def test_exchange_plan_executed_with_virtual_ranks(oracle_mod, binding, d, b, steady, tail, v_scale):
    """The whole consumer-side pipeline on one device, driven by sparsp_exchange_plan: every virtual rank starts
    from its own blocks, then, round by round and chunk by chunk in the plan's order, "fetches" exactly the plan's
    byte ranges of its packed buffer into a receive buffer that is NaN everywhere else (a device-to-device copy
    stands in for the peer copy of Section 6), runs the packed-source attention on that hop and merges.  K and V
    of blocks the rank does not own are NaN throughout.  The result must be the rank's rows of one-shot attention."""
    from paper_2609_32197_b200 import synth
    H, P = 4, 4
    wl = synth.Workload("xchg", H, d, (5, 11, 13), 70, b, 5 if b == 128 else 9, None, P, seed=71)
    Q, K, V = synth.make_qkv(wl, "cpu")
    V = (V.float() * v_scale).to(torch.bfloat16)  # 1: the generator's own V ~ N(0,1); 0.5: an extra case
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    ws = binding.make_workspace(shape, P)
    ref = oracle_mod.block_mask(Q, K, b, wl.topk_abs, wl.n_text)
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.topk_abs, ws)
    rank = np.array([(j * 3 + j // 4) % P for j in range(NB)], np.int32)
    rank_d = torch.as_tensor(rank).cuda()
    dg = pu.gpu_demand_pack(binding, shape, mo["mask"], rank_d, P, 0, Kd, Vd, ws)
    plan = binding.sparsp_exchange_plan(shape, P, dg["cnt"], dg["seg_offset"], steady, tail)
    entry = 2 * b * d * 2
    totals = dg["seg_total"][0].cpu().numpy()
    base = np.concatenate([[0], np.cumsum(totals)[:-1]]) * entry      # dense consumer bases of the packed buffer
    assert sum(t.n_bytes for t in plan) == int(dg["volume_bytes"].sum().item())
    o_ref, lse_ref = oracle_mod.attn_all(Q, K, V, ref["mask"], b)
    blk_of_tok = np.arange(N) // b
    hop = torch.empty_like(mo["mask"])
    nan_byte = 0xFF  # 0xFFFF is a bf16 NaN
    for r in range(P):
        foreign = torch.as_tensor(rank[blk_of_tok] != r)
        Kp, Vp = K.clone(), V.clone()
        Kp[:, foreign] = float("nan")
        Vp[:, foreign] = float("nan")
        Kpd, Vpd = Kp.cuda(), Vp.cuda()
        recv = torch.full_like(dg["packed"], nan_byte)
        acc = torch.zeros_like(Qd)
        acc_lse = torch.full((1, H, N), float("-inf"), dtype=torch.float32, device="cuda")
        binding.sparsp_hop_mask(shape, mo["mask"], rank_d, P, r, r, hop)          # local blocks first
        binding.sparsp_sparse_attn_fwd(shape, Qd, Kpd, Vpd, hop, 0.0, acc, acc_lse, ws)
        mine = [t for t in plan if t.consumer == r]
        for k in range(P - 1):
            chunks = [t for t in mine if t.round == k]
            assert [t.order for t in chunks] == list(range(len(chunks)))
            p = chunks[0].producer
            assert p == (r - (k + 1)) % P
            rows_t = torch.as_tensor(np.repeat(rank == r, b)[:N]).cuda()
            for t in chunks:
                # Fetch: exactly the planned byte range, nothing else ...
                lo = int(base[r]) + t.byte_offset
                recv[lo:lo + t.n_bytes].copy_(dg["packed"][lo:lo + t.n_bytes])
                # ... and attention on the chunk as soon as it is there (Section 7.1), before the next one arrives
                binding.sparsp_hop_chunk_mask(shape, mo["mask"], rank_d, P, r, p, t.head_begin, t.head_end, hop)
                assert np.array_equal(pu.u32(hop[0]),
                                      oracle_mod.hop_mask(ref["mask"], rank, r, p, t.head_begin, t.head_end))
                part = torch.zeros_like(Qd)
                part_lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
                binding.sparsp_sparse_attn_fwd_packed(shape, Qd, Kpd, Vpd, hop, rank_d, P, r, dg["union_mask"],
                                                      dg["seg_offset"], dg["seg_total"], recv, recv.numel() - 64,
                                                      None, 0.0, part, part_lse, ws)
                part[:, ~rows_t] = 0                      # rows of other ranks are left unwritten by the call
                part_lse[0][:, ~rows_t] = float("-inf")
                binding.sparsp_attn_merge(shape, acc, acc_lse, part, part_lse, acc, acc_lse)
        torch.cuda.synchronize()
        assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
        rows = np.repeat(rank == r, b)[:N]
        got = acc.float().cpu().numpy()[:, rows]
        assert np.isfinite(got).all()
        err = np.abs(got - o_ref[:, rows])
        tol_max = pu.ATTN_MAX_ABS + P * 2.0 ** -9 * np.abs(o_ref[:, rows]).max()
        tol_mean = pu.ATTN_MEAN_ABS + P * 2.0 ** -10 * np.abs(o_ref[:, rows]).mean()
        assert err.max() <= tol_max and err.mean() <= tol_mean, (r, err.max(), err.mean())
        assert np.abs(acc_lse[0].cpu().numpy()[:, rows] - lse_ref[:, rows]).max() < 2e-2
