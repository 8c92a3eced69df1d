"""Pins for the oracle's placement tools: the block permutation (Section 4.3), the token permutation and
its inverse, and the remote-K sharing statistic (Section 3.2) against the band-mask closed form."""
import numpy as np
import torch


def _mask_from_bool(M):
    H, NB, _ = M.shape
    out = np.zeros((H, NB, (NB + 31) // 32), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in range(NB):
                if M[h, i, j]:
                    out[h, i, j >> 5] |= np.uint32(1 << (j & 31))
    return out


def test_permutation_is_a_bijection_grouped_by_rank(oracle_mod):
    rng = np.random.default_rng(0)
    for NB, P, b, tail in [(10, 3, 64, 0), (37, 4, 128, 11), (8, 8, 64, 63), (5, 1, 64, 1)]:
        N = NB * b - tail
        rank = rng.integers(0, P, NB).astype(np.int32)
        bos, off, first = oracle_mod.placement_permutation(rank, P, N, b)
        assert sorted(bos.tolist()) == list(range(NB))                       # bijection
        assert off[0] == 0 and off[-1] == N
        for r in range(P):
            seg = bos[first[r]:first[r + 1]]
            assert np.all(rank[seg] == r) and np.all(np.diff(seg) > 0)       # grouped by rank, ascending inside
        sizes = np.diff(off)
        assert np.all(sizes == np.minimum(b, N - bos.astype(np.int64) * b))


def test_token_permutation_round_trip_and_block_membership(oracle_mod):
    rng = np.random.default_rng(1)
    H, b, d, NB, P = 2, 64, 8, 7, 3
    N = NB * b - 20
    X = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    rank = np.array([2, 0, 1, 1, 0, 2, 0], np.int32)
    bos, off, first = oracle_mod.placement_permutation(rank, P, N, b)
    Y = oracle_mod.permute_tokens(X, bos, off, b)
    assert torch.equal(oracle_mod.permute_tokens(Y, bos, off, b, inverse=True), X)
    # rank 0 owns logical blocks 1, 4, 6 (the last one ragged): its part of Y is exactly those, in that order
    want = torch.cat([X[:, 1 * b:2 * b], X[:, 4 * b:5 * b], X[:, 6 * b:N]], dim=1)
    assert torch.equal(Y[:, :want.shape[1]], want)
    assert first.tolist() == [0, 3, 5, 7]


def test_sharing_histogram_bruteforce_and_band_closed_form(oracle_mod):
    # (a) tiny brute force, written differently: per (r, h, j) set arithmetic
    rng = np.random.default_rng(2)
    H, NB, P = 2, 12, 3
    M = rng.random((H, NB, NB)) < 0.3
    rank = rng.integers(0, P, NB).astype(np.int32)
    hist = oracle_mod.sharing_histogram(_mask_from_bool(M), rank, P)
    for r in range(P):
        local = np.flatnonzero(rank == r)
        want = np.zeros(101, np.int64)
        for h in range(H):
            cnt = M[h][local].sum(0)
            for j in np.flatnonzero((rank != r) & (cnt > 0)):
                want[(100 * int(cnt[j])) // len(local)] += 1
        assert np.array_equal(hist[r], want)
    # (b) Section 4.3's band mask under the interval-periodic layout: the halo block at distance e from the
    # interval (e = 1..delta) is accessed by (delta - e + 1) of the L local positions in every frame
    T, B, G, delta, b = 4, 20, 4, 3, 64
    NB = T * B
    Mb = np.zeros((1, NB, NB), bool)
    for t in range(T):
        for s in range(B):
            for t2 in range(T):
                for s2 in range(max(0, s - delta), min(B, s + delta + 1)):
                    Mb[0, t * B + s, t2 * B + s2] = True
    rank = oracle_mod.placement_periodic(NB, G, b, B * b, NB * b)
    hist = oracle_mod.sharing_histogram(_mask_from_bool(Mb), rank, G)
    L = B // G
    for r in range(G):
        want = np.zeros(101, np.int64)
        sides = (1 if r > 0 else 0) + (1 if r < G - 1 else 0)
        for e in range(1, delta + 1):
            want[(100 * (delta - e + 1) * T) // (L * T)] += sides * T      # one halo block per side per frame
        assert np.array_equal(hist[r], want), (r, hist[r].nonzero(), want.nonzero())
