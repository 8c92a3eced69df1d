"""Pins for the oracle's step 3 (block-sparse attention): library SDPA in fp64 (dense and with a
token-level Boolean mask), special cases with closed forms, and agreement of the two oracle forms."""
import numpy as np
import torch
import torch.nn.functional as F


def _rand_qkv(rng, H, N, d, scale=1.0):
    mk = lambda: torch.tensor(rng.standard_normal((H, N, d)) * scale, dtype=torch.float32).to(torch.bfloat16)
    return mk(), mk(), mk()


def _mask_words(M):
    H, NB, _ = M.shape
    Wd = (NB + 31) // 32
    out = np.zeros((H, NB, Wd), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in range(NB):
                if M[h, i, j]:
                    out[h, i, j >> 5] |= np.uint32(1 << (j & 31))
    return out


def _sdpa64(Q, K, V, token_mask=None):
    q, k, v = (x.to(torch.float64).unsqueeze(0) for x in (Q, K, V))
    am = None if token_mask is None else torch.tensor(token_mask).unsqueeze(0)
    return F.scaled_dot_product_attention(q, k, v, attn_mask=am)[0].numpy()


def test_all_ones_mask_equals_dense_attention(oracle_mod):
    rng = np.random.default_rng(0)
    H, b, d = 2, 64, 32
    N = 3 * b + 17
    NB = 4
    Q, K, V = _rand_qkv(rng, H, N, d)
    M = np.ones((H, NB, NB), bool)
    out, lse = oracle_mod.attn_all(Q, K, V, _mask_words(M), b)
    ref = _sdpa64(Q, K, V)
    assert np.abs(out - ref).max() < 1e-6
    # log-sum-exp against an independent fp64 computation
    s = torch.einsum("hqc,hkc->hqk", Q.double(), K.double()) / np.sqrt(d)
    assert np.abs(lse - torch.logsumexp(s, dim=-1).numpy()).max() < 1e-5


def test_block_mask_equals_sdpa_with_token_mask(oracle_mod):
    rng = np.random.default_rng(1)
    H, b, d = 3, 64, 16
    N = 4 * b + 5
    NB = 5
    Q, K, V = _rand_qkv(rng, H, N, d, 1.5)
    M = rng.random((H, NB, NB)) < 0.4
    for i in range(NB):
        M[:, i, i] = True
    blk = np.arange(N) // b
    tok = M[:, blk][:, :, blk]  # [H][N][N]
    out, _ = oracle_mod.attn_all(Q, K, V, _mask_words(M), b)
    ref = _sdpa64(Q, K, V, tok)
    assert np.abs(out - ref).max() < 1e-6


def test_dense_masked_form_agrees_and_rows_sum_to_one(oracle_mod):
    rng = np.random.default_rng(2)
    H, b, d = 2, 64, 64
    N = 2 * b + 40
    NB = 3
    Q, K, V = _rand_qkv(rng, H, N, d)
    M = rng.random((H, NB, NB)) < 0.5
    M[:, :, 0] = True
    words = _mask_words(M)
    a, _ = oracle_mod.attn_all(Q, K, V, words, b)
    bb, rowsum = oracle_mod.attn_dense_masked(Q, K, V, words, b)
    assert np.abs(a - bb).max() < 1e-6
    assert np.abs(rowsum - 1.0).max() < 1e-12


def test_single_kept_block_constant_v_and_zero_q(oracle_mod):
    rng = np.random.default_rng(3)
    H, b, d, NB = 1, 64, 8, 4
    N = NB * b - 9
    Q, K, V = _rand_qkv(rng, H, N, d)
    # (a) only block 2 kept, V constant on block 2 -> output equals that constant
    V2 = V.clone()
    V2[0, 2 * b:3 * b] = 0.75
    M = np.zeros((H, NB, NB), bool)
    M[:, :, 2] = True
    out, _ = oracle_mod.attn_all(Q, K, V2, _mask_words(M), b)
    assert np.abs(out - 0.75).max() < 1e-7
    # (b) Q = 0 -> uniform weights -> mean of V over the kept valid tokens (ragged block included)
    M = np.zeros((H, NB, NB), bool)
    M[:, :, 1] = True
    M[:, :, 3] = True
    out, lse = oracle_mod.attn_all(torch.zeros_like(Q), K, V, _mask_words(M), b)
    kept = torch.cat([V[0, b:2 * b], V[0, 3 * b:N]]).double()
    assert np.abs(out[0] - kept.mean(0).numpy()).max() < 1e-6
    assert np.abs(lse - np.log(len(kept))).max() < 1e-6


def test_explicit_scale_and_sampled_units(oracle_mod):
    rng = np.random.default_rng(4)
    H, b, d, NB = 2, 64, 16, 3
    N = NB * b
    Q, K, V = _rand_qkv(rng, H, N, d)
    M = np.ones((H, NB, NB), bool)
    words = _mask_words(M)
    full, _ = oracle_mod.attn_all(Q, K, V, words, b, scale=0.3)
    q = Q.double() * (0.3 * np.sqrt(d))  # SDPA divides by sqrt(d)
    ref = F.scaled_dot_product_attention(q.unsqueeze(0), K.double().unsqueeze(0), V.double().unsqueeze(0))[0].numpy()
    assert np.abs(full - ref).max() < 1e-6
    part, _ = oracle_mod.attn_rows(Q, K, V, words, b, [(1, 2), (0, 0)], scale=0.3)
    assert np.array_equal(part[0], full[1, 2 * b:3 * b])
    assert np.array_equal(part[1], full[0, 0:b])


def test_hop_partials_merge_to_full_attention(oracle_mod):
    """Ring-style decomposition: attention of a consumer rank over each producer's blocks separately,
    merged by log-sum-exp, equals attention over all kept blocks at once (and library SDPA)."""
    rng = np.random.default_rng(6)
    H, b, d, NB, P = 2, 64, 16, 6, 3
    N = NB * b - 11
    Q, K, V = _rand_qkv(rng, H, N, d)
    M = rng.random((H, NB, NB)) < 0.5
    for i in range(NB):
        M[:, i, i] = True
    words = _mask_words(M)
    rank = np.array([0, 1, 2, 2, 0, 1], np.int32)
    full, full_lse = oracle_mod.attn_all(Q, K, V, words, b)
    for r in range(P):
        acc = np.zeros_like(full)
        acc_lse = np.full(full_lse.shape, -np.inf, np.float32)
        for p in range(P):
            hm = oracle_mod.hop_mask(words, rank, r, p)
            # brute-force check of the hop mask definition
            for h in range(H):
                for i in range(NB):
                    for j in range(NB):
                        bit = (int(hm[h, i, j >> 5]) >> (j & 31)) & 1
                        assert bit == int(M[h, i, j] and rank[i] == r and rank[j] == p)
            # the chunks of a hop (head ranges) are disjoint and add up to the hop
            parts = [oracle_mod.hop_mask(words, rank, r, p, h0, h0 + 1) for h0 in range(H)]
            assert all(not pc[np.arange(H) != h0].any() for h0, pc in enumerate(parts))
            assert np.array_equal(np.bitwise_or.reduce(np.stack(parts)), hm)
            part, part_lse = oracle_mod.attn_all(Q, K, V, hm, b)
            acc, acc_lse = oracle_mod.attn_merge(acc, acc_lse, part, part_lse)
        rows = np.repeat(rank == r, b)[:N]
        assert np.abs(acc[:, rows] - full[:, rows]).max() < 1e-5
        assert np.abs(acc_lse[:, rows] - full_lse[:, rows]).max() < 1e-5
        assert np.all(acc_lse[:, ~rows] == -np.inf) and not acc[:, ~rows].any()


def test_merge_special_cases(oracle_mod):
    oa = np.array([[1.0, 2.0], [3.0, 4.0], [0.0, 0.0]], np.float32)
    ob = np.array([[5.0, 6.0], [7.0, 8.0], [0.0, 0.0]], np.float32)
    la = np.array([0.0, -np.inf, -np.inf], np.float32)
    lb = np.array([0.0, 2.0, -np.inf], np.float32)
    out, lse = oracle_mod.attn_merge(oa, la, ob, lb)
    assert np.allclose(out[0], [3.0, 4.0]) and np.isclose(lse[0], np.log(2.0))   # equal weights: mean
    assert np.allclose(out[1], [7.0, 8.0]) and lse[1] == 2.0                      # empty part a
    assert not out[2].any() and lse[2] == -np.inf                                 # both empty
