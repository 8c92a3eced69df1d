"""Pins for the oracle's step 1 (pool, score, top-k): closed forms, brute force, special cases.

None of these re-type the oracle's own loop: each expected value comes from exact integer
arithmetic, a closed form, or an independent brute-force enumeration.
"""
import numpy as np
import torch


def _bf16(a):
    return torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)


def _bits(mask_row, NB):
    return [j for j in range(NB) if (int(mask_row[j >> 5]) >> (j & 31)) & 1]


# ----------------------------------------------------------------------------- pool
def test_pool_integer_inputs_closed_form(oracle_mod):
    # token t of block i, channel c holds (t mod 5) + c - i: integers, every partial sum exact.
    H, b, NB, d = 2, 64, 3, 8
    N = NB * b
    x = np.zeros((H, N, d), np.float32)
    for h in range(H):
        for n in range(N):
            for c in range(d):
                x[h, n, c] = (n % b) % 5 + c - (n // b) + h
    got = oracle_mod.pool(_bf16(x), b)
    # sum over t=0..63 of (t mod 5) = 12 full cycles * 10 + (0+1+2+3) = 126
    for h in range(H):
        for i in range(NB):
            for c in range(d):
                assert got[h, i, c] == np.float32(126 + 64 * (c - i + h)) / np.float32(64)


def test_pool_constant_block_and_ragged_tail(oracle_mod):
    b, d = 64, 4
    N = 64 + 10  # second block has 10 valid tokens
    x = np.full((1, N, d), 3.0, np.float32)
    x[0, 64:, 1] = np.arange(10)  # 0..9 -> mean 4.5
    x[0, 64:, 2] = -2.0
    got = oracle_mod.pool(_bf16(x), b)
    assert got.shape == (1, 2, d)
    assert np.all(got[0, 0] == 3.0)
    assert got[0, 1, 0] == 3.0 and got[0, 1, 1] == 4.5 and got[0, 1, 2] == -2.0


def test_pool_is_fp32_sequential_not_fp64(oracle_mod):
    # 1 then 63 copies of 2^-9: every fp32 add is exact here (needs 10 bits), so the mean is
    # exactly (1 + 63*2^-9)/64; and a second column where fp32 sequential order matters:
    # 2^24 followed by 63 ones stays 2^24 in fp32 sequential summation (each +1 is lost)...
    b, d = 64, 2
    x = np.zeros((1, b, d), np.float32)
    x[0, 0, 0] = 1.0
    x[0, 1:, 0] = 2.0 ** -9
    # bf16 cannot hold 2^24+1 anyway; use 2^8 * 2^16: big = 2^24 is exact in bf16
    x[0, 0, 1] = 2.0 ** 24
    x[0, 1:, 1] = 1.0
    got = oracle_mod.pool(_bf16(x), b)
    assert got[0, 0, 0] == np.float32((1 + 63 * 2.0 ** -9) / 64)
    assert got[0, 0, 1] == np.float32(2.0 ** 24 / 64)  # ascending-token fp32 chain loses the ones


# ----------------------------------------------------------------------------- score + top-k
def _exact_construction(NB, b, d):
    """Q block i = (2i, -1, -16, -256, 0...), K block j = (j, d0, d1, d2, 0...) with
    j^2 = d0 + 16 d1 + 256 d2  =>  S[i][j] = 2ij - j^2 = i^2 - (i-j)^2 exactly."""
    N = NB * b
    q = np.zeros((1, N, d), np.float32)
    k = np.zeros((1, N, d), np.float32)
    for j in range(NB):
        sq = j * j
        q[0, j * b:(j + 1) * b, :4] = [2 * j, -1, -16, -256]
        k[0, j * b:(j + 1) * b, :4] = [j, sq % 16, (sq // 16) % 16, sq // 256]
    return _bf16(q), _bf16(k)


def test_scores_exact_integer_construction(oracle_mod):
    NB, b, d = 40, 64, 8
    q, k = _exact_construction(NB, b, d)
    sc = oracle_mod.scores(oracle_mod.pool(q, b), oracle_mod.pool(k, b))
    for i in range(NB):
        for j in range(NB):
            assert sc[0, i, j] == float(i * i - (i - j) * (i - j))


def test_topk_nearest_blocks_with_lower_index_tiebreak(oracle_mod):
    NB, b, d = 40, 64, 8
    q, k = _exact_construction(NB, b, d)
    for kk in (1, 2, 5, 8, 39, 40):
        res = oracle_mod.block_mask(q, k, b, kk)
        for i in range(NB):
            # closed form: sort by (|i-j|, j) and keep kk  (ties |i-j| equal -> lower j first)
            expect = sorted(sorted(range(NB), key=lambda j: (abs(i - j), j))[:kk])
            assert _bits(res["mask"][0, i], NB) == expect, (kk, i)
            assert list(res["kv_list"][0, i, :kk]) == expect
            assert res["kv_count"][0, i] == kk


def test_topk_equals_block_count_gives_all_ones(oracle_mod):
    rng = np.random.default_rng(0)
    NB, b, d, H = 37, 64, 16, 3
    N = NB * b - 20
    q = _bf16(rng.standard_normal((H, N, d)))
    k = _bf16(rng.standard_normal((H, N, d)))
    res = oracle_mod.block_mask(q, k, b, NB)
    for h in range(H):
        for i in range(NB):
            assert _bits(res["mask"][h, i], NB) == list(range(NB))
    # bits beyond NB in the last word stay clear
    assert int(res["mask"][0, 0, 1]) >> (NB - 32) == 0


def test_top1_one_hot_blocks_identity(oracle_mod):
    NB, b, d = 16, 64, 16
    x = np.zeros((1, NB * b, d), np.float32)
    for j in range(NB):
        x[0, j * b:(j + 1) * b, j] = 1.0
    res = oracle_mod.block_mask(_bf16(x), _bf16(x), b, 1)
    for i in range(NB):
        assert _bits(res["mask"][0, i], NB) == [i]


def test_topk_matches_bruteforce_sort_small(oracle_mod):
    rng = np.random.default_rng(1)
    NB, H = 8, 4
    sc = rng.integers(-3, 4, size=(H, NB, NB)).astype(np.float32)  # many exact ties
    sc[0, 0, 2] = -0.0
    sc[0, 0, 5] = 0.0
    is_text = np.zeros(NB, np.uint8)
    for kk in range(1, NB + 1):
        mask, kv_list, kv_count = oracle_mod.topk_mask(sc, is_text, kk)
        for h in range(H):
            for i in range(NB):
                order = sorted(range(NB), key=lambda j: (-float(sc[h, i, j]), j))
                assert _bits(mask[h, i], NB) == sorted(order[:kk])
                assert kv_count[h, i] == kk


def test_text_blocks_forced_and_excluded_from_candidates(oracle_mod):
    rng = np.random.default_rng(2)
    NB, H = 12, 2
    sc = rng.standard_normal((H, NB, NB)).astype(np.float32)
    sc[:, :, 10:] = 100.0  # text blocks have the top scores but must not use up k
    is_text = np.zeros(NB, np.uint8)
    is_text[10:] = 1
    mask, kv_list, kv_count = oracle_mod.topk_mask(sc, is_text, 3)
    for h in range(H):
        for i in range(NB):
            order = sorted(range(10), key=lambda j: (-float(sc[h, i, j]), j))
            assert _bits(mask[h, i], NB) == sorted(order[:3]) + [10, 11]
            assert kv_count[h, i] == 5


def test_text_block_flags_and_resolve_topk(oracle_mod):
    # 17550 video + 226 text tokens, b = 64: 274 pure video blocks, block 274 is mixed
    flags = oracle_mod.text_block_flags(17550, 226, 64)
    assert len(flags) == 278 and flags[:274].sum() == 0 and flags[274:].sum() == 4
    assert oracle_mod.resolve_topk(15, 384) == 58
    assert oracle_mod.resolve_topk(20, 274) == 55
    assert oracle_mod.resolve_topk(10, 591) == 60
    assert [oracle_mod.resolve_topk(p, 929) for p in (5, 10, 25)] == [47, 93, 233]
    assert oracle_mod.resolve_topk(0, 10) == 1 and oracle_mod.resolve_topk(100, 10) == 10


def test_fp32_scores_close_to_fp64_scores(oracle_mod):
    rng = np.random.default_rng(3)
    pq = rng.standard_normal((2, 9, 128)).astype(np.float32)
    pk = rng.standard_normal((2, 9, 128)).astype(np.float32)
    s32 = oracle_mod.scores(pq, pk)
    s64 = oracle_mod.scores_f64(pq, pk)
    ref = np.einsum("hic,hjc->hij", pq.astype(np.float64), pk.astype(np.float64))
    assert np.allclose(s64, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(s32, ref, rtol=1e-5, atol=1e-5)
