"""GPU parity tests (small sizes): the three C-ABI calls against the CPU oracle, element by element.
Sizes are chosen so that the oracle finishes in seconds yet every kernel runs several tiles and a
ragged tail; both memory layouts and every supported (head_dim, block) pair are covered."""
import numpy as np
import pytest
import torch

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32197_b200 import binding as b
    b.lib()  # raises if the CUDA library is missing: there is no fallback
    assert torch.cuda.is_available()
    return b


def _gen(wl):
    from paper_2609_32197_b200 import synth
    return synth.make_qkv(wl, "cpu")


def _workload(name, heads, d, grid, n_text, b, k, ranks, seed=0):
    from paper_2609_32197_b200 import synth
    return synth.Workload(name, heads, d, grid, n_text, b, k, None, ranks, seed=seed)


def _run_all(oracle, binding, wl, rank_np, layout="HND", include_local=False, full_attn=True, lse=True):
    Q, K, V = _gen(wl)
    H, N, d = Q.shape
    b, P, k = wl.block, wl.ranks, wl.topk_abs
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    Qd, Kd, Vd = (pu.to_layout(x.cuda(), layout) for x in (Q, K, V))
    ws = binding.make_workspace(shape, P)
    # step 1
    ref, got = pu.check_mask(oracle, binding, shape, Q, K, Qd, Kd, k, wl.n_text, ws)
    # step 2
    rank_d = torch.as_tensor(rank_np, dtype=torch.int32).cuda()
    flags = binding.SPARSP_INCLUDE_LOCAL if include_local else 0
    dg = pu.gpu_demand_pack(binding, shape, got["mask"], rank_d, P, flags, Kd, Vd, ws)
    dref = pu.check_demand(oracle, binding, shape, ref["mask"], rank_np, P, include_local, dg)
    packed_ref = oracle.pack(K, V, dref["U"], rank_np, b, P, dref["total"], include_local=include_local)
    packed = dg["packed"].cpu().numpy()
    assert np.array_equal(packed[:packed_ref.size], packed_ref), "packed bytes"
    assert (packed[packed_ref.size:] == 0xAB).all(), "wrote past the end"
    # step 3
    Od = torch.zeros_like(Qd)
    lse_d = torch.zeros(1, H, N, dtype=torch.float32, device="cuda") if lse else None
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, got["mask"], 0.0, Od, lse_d, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    NB = wl.n_blocks
    units = [(h, i) for h in range(H) for i in range(NB)] if full_attn else pu.sample_units(H, NB, rank_np, 8, 0)
    return pu.check_attn_units(oracle, Q, K, V, ref["mask"], b, pu.from_layout(Od, layout), units,
                               lse_gpu=None if lse_d is None else lse_d[0])


def test_tiny_config_full(oracle_mod, binding):
    from paper_2609_32197_b200 import synth
    wl = synth.WORKLOADS["tiny"]
    rank = oracle_mod.placement_contiguous(wl.n_blocks, wl.ranks)
    mx, mean = _run_all(oracle_mod, binding, wl, rank)
    print(f"tiny: attn max abs {mx:.3e} mean abs {mean:.3e}")


@pytest.mark.parametrize("d,b", [(64, 64), (128, 64), (64, 128), (128, 128)])
@pytest.mark.parametrize("layout", ["HND", "NHD"])
def test_ragged_text_all_shapes(oracle_mod, binding, d, b, layout):
    # 5*11*13 = 715 video + 70 text = 785 tokens: ragged last block for both block sizes, text tail
    wl = _workload("ragged", 3, d, (5, 11, 13), 70, b, 3 if b == 128 else 5, 3, seed=3)
    rank = np.array([(j * 5) % 3 for j in range(wl.n_blocks)], np.int32)  # scattered placement
    _run_all(oracle_mod, binding, wl, rank, layout=layout, include_local=(layout == "NHD"))


def test_multi_word_masks_and_periodic_placement(oracle_mod, binding):
    # 4*24*32 = 3072 tokens, block 64 -> 48 blocks (2 mask words), frames aligned to blocks
    wl = _workload("multiword", 4, 64, (4, 24, 32), 0, 64, 7, 4, seed=5)
    rank = oracle_mod.placement_periodic(wl.n_blocks, 4, 64, wl.frame_tokens, wl.n_video)
    shape = binding.make_shape(4, 64, wl.grid, 0, 64)
    assert np.array_equal(binding.sparsp_placement_periodic(shape, 4).numpy(), rank)
    assert np.array_equal(binding.sparsp_placement_contiguous(shape, 4).numpy(),
                          oracle_mod.placement_contiguous(wl.n_blocks, 4))
    _run_all(oracle_mod, binding, wl, rank)


def test_exact_ties_lowest_index_wins(oracle_mod, binding):
    """Integer construction with S[i][j] = i^2 - (i-j)^2: every row has exact score ties."""
    NB, b, d, H = 40, 64, 64, 2
    N = NB * b
    q = np.zeros((H, N, d), np.float32)
    k = np.zeros((H, N, d), np.float32)
    for j in range(NB):
        sq = j * j
        q[:, j * b:(j + 1) * b, :4] = [2 * j, -1, -16, -256]
        k[:, j * b:(j + 1) * b, :4] = [j, sq % 16, (sq // 16) % 16, sq // 256]
    Q, K = torch.tensor(q).to(torch.bfloat16), torch.tensor(k).to(torch.bfloat16)
    shape = binding.make_shape(H, d, (1, NB, b), 0, b)
    ws = binding.make_workspace(shape, 1)
    for kk in (1, 2, 6, 39, 40):
        ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Q.cuda(), K.cuda(), kk, 0, ws)
        row = pu.u32(got["mask"][0])[0, 20]
        bits = [j for j in range(NB) if (int(row[j >> 5]) >> (j & 31)) & 1]
        assert bits == sorted(sorted(range(NB), key=lambda j: (abs(20 - j), j))[:kk])


def test_signed_zero_scores_tie(oracle_mod, binding):
    """Q block 0 is all zeros with K mixing signs: scores are +0 and -0, which must compare equal."""
    NB, b, d, H = 8, 64, 64, 1
    N = NB * b
    rng = np.random.default_rng(0)
    k = rng.standard_normal((H, N, d)).astype(np.float32)
    q = rng.standard_normal((H, N, d)).astype(np.float32)
    q[:, :b] = 0.0
    q[:, :b:2, 0] = -0.0
    Q, K = torch.tensor(q).to(torch.bfloat16), torch.tensor(k).to(torch.bfloat16)
    shape = binding.make_shape(H, d, (1, NB, b), 0, b)
    ws = binding.make_workspace(shape, 1)
    ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Q.cuda(), K.cuda(), 3, 0, ws)
    assert list(ref["kv_list"][0, 0]) == [0, 1, 2]


def test_dense_mask_matches_library_sdpa(oracle_mod, binding):
    """top-k = NB keeps everything: the kernel must reproduce dense attention (library fp32 SDPA)."""
    wl = _workload("dense", 2, 128, (2, 12, 20), 0, 128, 4, 2, seed=9)  # 480 tokens -> 4 blocks (last: 96)
    Q, K, V = _gen(wl)
    shape = binding.make_shape(2, 128, wl.grid, 0, 128)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    got = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.n_blocks, ws)
    assert int(torch.bitwise_and(got["mask"], 0xF).eq(0xF).all())
    Od = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, got["mask"], 0.0, Od, None, ws)
    ref = torch.nn.functional.scaled_dot_product_attention(Qd.float()[None], Kd.float()[None], Vd.float()[None])[0]
    err = (Od.float() - ref).abs()
    assert err.max().item() <= pu.ATTN_MAX_ABS and err.mean().item() <= pu.ATTN_MEAN_ABS


def test_explicit_scale_single_rank_and_capacity_overflow(oracle_mod, binding):
    wl = _workload("cap", 2, 64, (2, 16, 16), 0, 64, 3, 2, seed=11)  # 512 tokens, 8 blocks
    Q, K, V = _gen(wl)
    shape = binding.make_shape(2, 64, wl.grid, 0, 64)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Qd, Kd, 3, 0, ws)
    # explicit softmax scale
    Od = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, got["mask"], 0.05, Od, None, ws)
    units = [(h, i) for h in range(2) for i in range(8)]
    pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], 64, Od, units, scale=0.05)
    # one rank: nothing is remote
    rank1 = torch.zeros(8, dtype=torch.int32, device="cuda")
    d1 = pu.gpu_demand_pack(binding, shape, got["mask"], rank1, 1, 0, Kd, Vd, ws)
    assert d1["total_entries"] == 0 and int(d1["volume_bytes"].sum()) == 0
    assert bool((d1["packed"] == 0xAB).all())
    # capacity one entry short: the last entry is skipped, nothing beyond capacity is touched
    rank2 = torch.as_tensor(oracle_mod.placement_contiguous(8, 2)).cuda()
    full = pu.gpu_demand_pack(binding, shape, got["mask"], rank2, 2, 0, Kd, Vd, ws)
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    n = full["total_entries"]
    short = pu.gpu_demand_pack(binding, shape, got["mask"], rank2, 2, 0, Kd, Vd, ws, capacity_entries=n - 1)
    assert binding.sparsp_status(ws) == binding.SPARSP_ERR_CAPACITY
    assert binding.sparsp_status(ws) == binding.SPARSP_OK  # reading resets it
    entry = 2 * 64 * 64 * 2
    assert torch.equal(short["packed"][:(n - 1) * entry], full["packed"][:(n - 1) * entry])
    assert bool((short["packed"][(n - 1) * entry:] == 0xAB).all())


def test_destination_bases(oracle_mod, binding):
    wl = _workload("bases", 2, 64, (2, 16, 16), 0, 64, 3, 2, seed=12)
    Q, K, V = _gen(wl)
    shape = binding.make_shape(2, 64, wl.grid, 0, 64)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Qd, Kd, 3, 0, ws)
    rank = oracle_mod.placement_contiguous(8, 2)
    dref = oracle_mod.demand(ref["mask"], rank, 2, 64, 64)
    entry = 2 * 64 * 64 * 2
    base = np.array([int(dref["total"][1]) * entry + 4096, 0], np.int64)  # swapped, with a gap
    expect = oracle_mod.pack(K, V, dref["U"], rank, 64, 2, dref["total"], dst_base=base)
    outs = binding.alloc_demand_outputs(shape, 2)
    packed = torch.zeros(expect.size, dtype=torch.uint8, device="cuda")
    binding.sparsp_demand_pack(shape, got["mask"], torch.as_tensor(rank).cuda(), 2, 0, Kd, Vd, outs["union_mask"],
                               outs["cnt"], outs["seg_offset"], outs["seg_total"], outs["volume_bytes"], packed,
                               expect.size, torch.as_tensor(base).cuda(), ws)
    torch.cuda.synchronize()
    assert np.array_equal(packed.cpu().numpy(), expect)


def test_invalid_arguments_are_rejected_on_the_host(binding):
    shape = binding.make_shape(2, 64, (2, 16, 16), 0, 64)
    ws = binding.make_workspace(shape, 2)
    x = torch.zeros(2, 512, 64, dtype=torch.bfloat16, device="cuda")
    outs = binding.alloc_mask_outputs(shape, 3)
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_block_mask(shape, x, x, 0, outs["mask"], None, None, None, None, ws)
    assert e.value.code == binding.SPARSP_ERR_INVALID_ARG
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_block_mask(shape, None, x, 3, outs["mask"], None, None, None, None, ws)
    assert e.value.code == binding.SPARSP_ERR_INVALID_ARG
    bad = binding.make_shape(2, 96, (2, 16, 16), 0, 64)
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_block_mask(bad, x, x, 3, outs["mask"], None, None, None, None, ws)
    assert e.value.code == binding.SPARSP_ERR_UNSUPPORTED
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_sparse_attn_fwd(shape, x, x, x, outs["mask"], -1.0, x, None, ws)
    assert e.value.code == binding.SPARSP_ERR_INVALID_ARG
    d = binding.alloc_demand_outputs(shape, 2)
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_demand_pack(shape, outs["mask"], torch.zeros(8, dtype=torch.int32, device="cuda"), 0, 0, x, x,
                                   d["union_mask"], d["cnt"], d["seg_offset"], d["seg_total"], d["volume_bytes"],
                                   x, 16, None, ws)
    assert e.value.code == binding.SPARSP_ERR_INVALID_ARG


def _stack_batches(xs, layout):
    """list of [H][N][d] CPU tensors -> device tensor [B][H][N][d] or [B][N][H][d]"""
    t = torch.stack(xs, 0).cuda()
    return t.contiguous() if layout == "HND" else t.permute(0, 2, 1, 3).contiguous()


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("v_scale", [1.0, 0.5])
def test_batch_of_two(oracle_mod, binding, layout, v_scale):
    """Batch is an independent outer dimension: each batch item must match the oracle run on it alone.
    v_scale = 1 is the generator's own V ~ N(0,1); 0.5 (exact in bf16) is an extra case with smaller outputs."""
    b, d, H, P, k = 64, 64, 2, 3, 4
    wls = [_workload("b0", H, d, (3, 9, 13), 40, b, k, P, seed=31), _workload("b1", H, d, (3, 9, 13), 40, b, k, P, seed=32)]
    data = [(Q, K, (V.float() * v_scale).to(torch.bfloat16)) for (Q, K, V) in (_gen(w) for w in wls)]
    N, NB = wls[0].n_tokens, wls[0].n_blocks
    shape = binding.make_shape(H, d, wls[0].grid, 40, b, batch=2, layout=layout)
    Qd, Kd, Vd = (_stack_batches([x[i] for x in data], layout) for i in range(3))
    ws = binding.make_workspace(shape, P)
    mo = binding.alloc_mask_outputs(shape, k, with_list=True, with_pooled=True)
    binding.sparsp_block_mask(shape, Qd, Kd, k, mo["mask"], mo["kv_list"], mo["kv_count"], mo["pooled_q"],
                              mo["pooled_k"], ws)
    rank = np.array([(j * 2) % P for j in range(NB)], np.int32)
    dg = pu.gpu_demand_pack(binding, shape, mo["mask"], torch.as_tensor(rank).cuda(), P, 0, Kd, Vd, ws)
    Od = torch.zeros_like(Qd)
    lse = torch.zeros(2, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mo["mask"], 0.0, Od, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    entry = 2 * b * d * 2
    packed = dg["packed"].cpu().numpy()
    cursor = 0
    for bi, (Q, K, V) in enumerate(data):
        ref = oracle_mod.block_mask(Q, K, b, k, 40)
        assert np.array_equal(pu.u32(mo["mask"][bi]), ref["mask"])
        assert np.array_equal(mo["kv_list"][bi].cpu().numpy(), ref["kv_list"])
        assert np.array_equal(mo["pooled_k"][bi].cpu().numpy().view(np.uint32), ref["pk"].view(np.uint32))
        dref = oracle_mod.demand(ref["mask"], rank, P, b, d)
        assert np.array_equal(pu.u32(dg["union_mask"][bi]), dref["U"])
        assert np.array_equal(dg["cnt"][bi].cpu().numpy(), dref["cnt"])
        assert np.array_equal(dg["seg_offset"][bi].cpu().numpy(), dref["seg_off"])
        assert np.array_equal(dg["volume_bytes"][bi].cpu().numpy(), dref["volume"])
        pref = oracle_mod.pack(K, V, dref["U"], rank, b, P, dref["total"])
        assert np.array_equal(packed[cursor:cursor + pref.size], pref), f"packed bytes of batch item {bi}"
        cursor += pref.size
        O_b = Od[bi] if layout == "HND" else Od[bi].permute(1, 0, 2)
        units = [(h, i) for h in range(H) for i in range(NB)]
        pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], b, O_b, units, lse_gpu=lse[bi])
    assert (packed[cursor:] == 0xAB).all()


def test_degenerate_shapes(oracle_mod, binding):
    """One block only; k = 1; a virtual rank that owns nothing; odd block count with block = 128."""
    # (a) a single ragged block: NB = 1, k = 1, P = 2 (rank 1 owns nothing)
    wl = _workload("one", 2, 128, (1, 5, 9), 0, 128, 1, 2, seed=41)  # 45 tokens
    _run_all(oracle_mod, binding, wl, np.zeros(1, np.int32))
    # (b) k = 1 on several blocks, odd NB with block 128 (the last CTA holds a single query block)
    wl = _workload("odd", 2, 64, (3, 10, 21), 0, 128, 1, 4, seed=42)  # 630 tokens -> 5 blocks
    _run_all(oracle_mod, binding, wl, np.array([0, 0, 2, 2, 3], np.int32))  # rank 1 owns nothing
    # (c) odd NB with block 64: the last stacked Q tile has an empty lower half
    wl = _workload("odd64", 2, 128, (3, 10, 21), 0, 64, 2, 2, seed=43)  # 630 tokens -> 10 blocks ... use 9
    wl = _workload("odd64", 2, 128, (3, 9, 21), 0, 64, 2, 2, seed=43)  # 567 tokens -> 9 blocks
    _run_all(oracle_mod, binding, wl, oracle_mod.placement_contiguous(9, 2))


@pytest.mark.parametrize("d,b", [(128, 128), (64, 64), (128, 64)])
@pytest.mark.parametrize("jump", [30.0, 100.0])
def test_scores_far_above_the_first_tile(oracle_mod, binding, d, b, jump):
    """The kernel skips a tile's row-maximum pass when a norm bound shows the scores stay within 2^64 of the
    row's reference.  Here the first kept block scores 0 and a later one `jump` (log2 units) higher: 30 stays
    inside the bound (exponentials up to 2^30 against the old reference), 100 does not (reference must move).
    Both must give the oracle's result: the mean of V over the high-scoring block, to 2^-jump."""
    H = 2
    NB = 6
    N = NB * b - 5                                   # ragged last block
    rng = np.random.default_rng(17)
    scale_log2 = 1.4426950408889634 / np.sqrt(d)
    a = 4.0
    bb = jump / (a * scale_log2)                     # a * bb * scale * log2(e) = jump; both exact enough in bf16
    Q = torch.zeros(H, N, d, dtype=torch.bfloat16)
    K = torch.zeros(H, N, d, dtype=torch.bfloat16)
    Q[:, :, 0] = a
    Q[:, :, 1:] = torch.tensor(rng.standard_normal((H, N, d - 1)) * 0.05).to(torch.bfloat16)
    K[:, :, 1:] = torch.tensor(rng.standard_normal((H, N, d - 1)) * 0.05).to(torch.bfloat16)
    K[:, 3 * b:4 * b, 0] = bb                        # block 3 scores `jump` above the others
    V = torch.tensor(rng.standard_normal((H, N, d))).to(torch.bfloat16)
    M = np.zeros((H, NB, NB), bool)
    M[:, :, 0] = True
    M[:, :, 1] = True
    M[:, :, 3] = True
    M[:, ::2, 5] = True                              # every other query block also keeps the ragged block
    words = np.zeros((H, NB, 1), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in range(NB):
                if M[h, i, j]:
                    words[h, i, 0] |= np.uint32(1 << j)
    shape = binding.make_shape(H, d, (1, 1, N), 0, b)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    mask_d = torch.as_tensor(words.view(np.int32)).cuda()
    O = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mask_d, 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(H) for i in range(NB)]
    pu.check_attn_units(oracle_mod, Q, K, V, words, b, O, units, lse_gpu=lse[0])
    # closed form: the high block dominates by 2^jump, so every row is the mean of V over block 3
    want = V[:, 3 * b:4 * b].float().mean(1)
    assert (O.float().cpu() - want[:, None, :]).abs().max() < 2e-2


@pytest.mark.parametrize("d,b", [(128, 128), (64, 128), (128, 64), (64, 64)])
@pytest.mark.parametrize("outlier", [False, True])
@pytest.mark.parametrize("v_sigma", [1.0, 0.5])
def test_long_lists_with_final_reference_and_ragged_tail(oracle_mod, binding, d, b, outlier, v_sigma):
    """Lists long enough (13 kept blocks per row, a different random set per row) that the kernel stops
    updating a row's reference once the item's largest key norm bounds all remaining scores, with the ragged
    last block of the sequence in every list.  With `outlier` one block holds keys of 40 times the norm
    (orthogonal to the queries, so its scores stay ordinary): the item-wide bound then fails while the
    per-tile bound holds for the other tiles, and the reference keeps being checked tile by tile."""
    H, NB = 2, 20
    N = NB * b - 37
    rng = np.random.default_rng(23 + d + b)
    Q = torch.tensor(rng.standard_normal((H, N, d))).to(torch.bfloat16)
    K = torch.tensor(rng.standard_normal((H, N, d))).to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d)) * v_sigma).to(torch.bfloat16)
    if outlier:
        Q[:, :, 0] = 0.0
        K[:, 7 * b:8 * b, 0] = 40.0 * np.sqrt(d)
    words = np.zeros((H, NB, 1), np.uint32)
    for h in range(H):
        for i in range(NB):
            keep = set(rng.choice(NB - 1, 12, replace=False).tolist()) | {NB - 1}
            if outlier:
                keep.add(7)
            for j in keep:
                words[h, i, 0] |= np.uint32(1 << j)
    shape = binding.make_shape(H, d, (1, 1, N), 0, b)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, torch.as_tensor(words.view(np.int32)).cuda(), 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(H) for i in range(NB)]
    pu.check_attn_units(oracle_mod, Q, K, V, words, b, O, units, lse_gpu=lse[0])


@pytest.mark.parametrize("b,tokens_grid", [(64, (10, 50, 128)), (128, (10, 100, 128))])
def test_attention_near_the_largest_block_count(oracle_mod, binding, b, tokens_grid):
    """NB = 1000 (the limit is 1024): mask rows of 32 words, the list buffers and the sort of a head's work items
    at their largest.  Sampled query blocks against the oracle; every other row finite and written."""
    from paper_2609_32197_b200 import synth
    H, d, k = 1, 64, 9
    wl = synth.Workload("big_nb", H, d, tokens_grid, 0, b, k, None, 2, seed=5)
    assert wl.n_blocks == 1000
    Qd, Kd, Vd = synth.make_qkv(wl, "cuda")
    Q, K, V = Qd.cpu(), Kd.cpu(), Vd.cpu()
    shape = binding.make_shape(H, d, wl.grid, 0, b)
    ws = binding.make_workspace(shape, 2)
    got = pu.gpu_block_mask(binding, shape, Qd, Kd, k, ws)
    ref = oracle_mod.block_mask(Q, K, b, k, 0)
    assert np.array_equal(pu.u32(got["mask"][0]), ref["mask"])
    Od = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, wl.n_tokens, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, got["mask"], 0.0, Od, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
    units = [(0, i) for i in (0, 1, 31, 32, 499, 500, 767, 998, 999)]
    pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], b, Od, units, lse_gpu=lse[0])
    assert bool(torch.isfinite(Od.float()).all())
    assert bool((Od.float().abs().amax(dim=-1) > 0).all())


def test_demand_plan_with_the_most_ranks_and_blocks(oracle_mod, binding):
    """64 virtual ranks (the limit) over 1000 blocks, scattered placement with one rank that owns nothing: the
    per-head union table is at its largest; plan only, every integer against the oracle."""
    H, NB, b, d, P = 2, 1000, 64, 64, 64
    rng = np.random.default_rng(3)
    M = rng.random((H, NB, NB)) < 0.004
    M[:, np.arange(NB), np.arange(NB)] = True
    bits = np.zeros((H, NB, 32 * 32), bool)
    bits[:, :, :NB] = M
    words = (bits.reshape(H, NB, 32, 32) * (1 << np.arange(32, dtype=np.uint64))).sum(-1).astype(np.uint32)
    rank = rng.integers(0, P - 1, NB).astype(np.int32)  # rank P-1 owns no block
    shape = binding.make_shape(H, d, (1, 1, NB * b), 0, b)
    ws = binding.make_workspace(shape, P)
    outs = binding.alloc_demand_outputs(shape, P)
    mask_d = torch.as_tensor(words.view(np.int32)).cuda()[None]
    binding.sparsp_demand_pack(shape, mask_d, torch.as_tensor(rank).cuda(), P, binding.SPARSP_PLAN_ONLY, None, None,
                               outs["union_mask"], outs["cnt"], outs["seg_offset"], outs["seg_total"],
                               outs["volume_bytes"], None, 0, None, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    pu.check_demand(oracle_mod, binding, shape, words, rank, P, False, outs)


@pytest.mark.parametrize("seed", [1, 2, 3, 4, 5, 6])
@pytest.mark.parametrize("v_sigma", [1.0, 0.5])
def test_random_norm_profiles(oracle_mod, binding, seed, v_sigma):
    """Random shapes with key blocks and query rows scaled by random factors (0.1 ... 20): tiles whose norm
    bound holds, tiles where it fails, references that become final early, late or never, all in one launch."""
    rng = np.random.default_rng(100 + seed)
    d = int(rng.choice([64, 128]))
    b = int(rng.choice([64, 128]))
    H = 2
    NB = int(rng.integers(18, 30))
    N = NB * b - int(rng.integers(0, b - 1))
    keep_n = int(rng.integers(6, 16))
    Qf = rng.standard_normal((H, N, d)) * np.exp(rng.uniform(np.log(0.1), np.log(4.0), (H, N, 1)))
    Kf = rng.standard_normal((H, N, d))
    for j in range(NB):
        Kf[:, j * b:(j + 1) * b] *= np.exp(rng.uniform(np.log(0.1), np.log(20.0 if j % 5 == 0 else 2.0)))
    Q = torch.tensor(Qf).to(torch.bfloat16)
    K = torch.tensor(Kf).to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d)) * v_sigma).to(torch.bfloat16)
    Wd = (NB + 31) // 32
    words = np.zeros((H, NB, Wd), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in rng.choice(NB, keep_n, replace=False):
                words[h, i, j >> 5] |= np.uint32(1 << (int(j) & 31))
    shape = binding.make_shape(H, d, (1, 1, N), 0, b)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, torch.as_tensor(words.view(np.int32)).cuda(), 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(H) for i in range(NB)]
    pu.check_attn_units(oracle_mod, Q, K, V, words, b, O, units, lse_gpu=lse[0])


@pytest.mark.parametrize("d,b", [(128, 128), (64, 64), (128, 64), (64, 128)])
@pytest.mark.parametrize("level", [30.0, 74.0])
def test_fixed_reference_at_the_edge_of_its_bound(oracle_mod, binding, d, b, level):
    """An item whose norm bound |q| |k| scale log2(e) stays under 2^80 runs on the fixed reference 0.  Here every score
    is about +level or -level (log2 units; 74 is just inside the bound): query blocks that keep only the low-scoring
    blocks work with exponentials around 2^-74 throughout, blocks that keep only the high ones with 2^+74, the rest
    with both at once.  All must give the oracle's rows (and log-sum-exp), which for the one-sided blocks are close
    to the mean of V over the kept keys."""
    H, NB = 2, 12
    N = NB * b - 7                                    # ragged last block
    rng = np.random.default_rng(29)
    scale_log2 = 1.4426950408889634 / np.sqrt(d)
    a = float(np.sqrt(level / scale_log2))            # |q| = |k| = a: a * a * scale * log2(e) = level
    Q = torch.zeros(H, N, d, dtype=torch.float32)
    K = torch.zeros(H, N, d, dtype=torch.float32)
    Q[:, :, 0] = a
    K[:, :, 0] = a
    for j in range(1, NB, 2):
        K[:, j * b:(j + 1) * b, 0] = -a               # odd key blocks score -level, even ones +level
    Q[:, :, 1:] = torch.tensor(rng.standard_normal((H, N, d - 1)) * 0.02)
    K[:, :, 1:] = torch.tensor(rng.standard_normal((H, N, d - 1)) * 0.02)
    Q, K = Q.to(torch.bfloat16), K.to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d))).to(torch.bfloat16)
    M = np.zeros((H, NB, NB), bool)
    for i in range(NB):
        if i % 3 == 0:
            M[:, i, 1::2] = True                      # low blocks only (six kept blocks: enough tiles for the fixed reference)
        elif i % 3 == 1:
            M[:, i, 0::2] = True                      # high blocks only
        else:
            M[:, i, :] = True                         # both
    words = np.zeros((H, NB, 1), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in range(NB):
                if M[h, i, j]:
                    words[h, i, 0] |= np.uint32(1 << j)
    shape = binding.make_shape(H, d, (1, 1, N), 0, b)
    ws = binding.make_workspace(shape, 2)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    mask_d = torch.as_tensor(words.view(np.int32)).cuda()
    O = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mask_d, 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(H) for i in range(NB)]
    pu.check_attn_units(oracle_mod, Q, K, V, words, b, O, units, lse_gpu=lse[0])
    got_lse = lse[0].cpu().numpy()
    ln2 = 0.6931471805599453
    assert got_lse[:, :b].max() < -(level - 12) * ln2          # low-only rows: every term is tiny, none was lost
    assert got_lse[:, b:2 * b].min() > (level - 12) * ln2      # high-only rows
