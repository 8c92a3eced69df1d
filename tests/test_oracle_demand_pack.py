"""Pins for the oracle's step 2 (demand, volume, offsets, pack): brute-force enumeration of the
set definitions, the paper's direct-delivery example, the band-mask closed form, invariants."""
import os

import numpy as np
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mask_from_bool(M):
    H, NB, _ = M.shape
    Wd = (NB + 31) // 32
    out = np.zeros((H, NB, Wd), np.uint32)
    for h in range(H):
        for i in range(NB):
            for j in range(NB):
                if M[h, i, j]:
                    out[h, i, j >> 5] |= np.uint32(1 << (j & 31))
    return out


def _bits(words, NB):
    return {j for j in range(NB) if (int(words[j >> 5]) >> (j & 31)) & 1}


def _bruteforce_demand(M, rank, P):
    """Literal enumeration of D[r][h][p] = { j | P(j)=p and exists i in Q_r: M[h][i][j]=1 }."""
    H, NB, _ = M.shape
    D = {}
    for r in range(P):
        for h in range(H):
            for p in range(P):
                D[r, h, p] = {j for j in range(NB) if rank[j] == p
                              and any(M[h, i, j] for i in range(NB) if rank[i] == r)}
    return D


def test_demand_matches_bruteforce_enumeration(oracle_mod):
    rng = np.random.default_rng(0)
    for (H, NB, P, dens) in [(2, 10, 3, 0.2), (3, 37, 4, 0.1), (1, 70, 8, 0.05), (2, 33, 1, 0.3)]:
        M = rng.random((H, NB, NB)) < dens
        rank = rng.integers(0, P, NB).astype(np.int32)
        b, d = 64, 128
        for incl in (False, True):
            res = oracle_mod.demand(_mask_from_bool(M), rank, P, b, d, include_local=incl)
            D = _bruteforce_demand(M, rank, P)
            for r in range(P):
                vol = 0
                cursor = 0
                for p in range(P):
                    for h in range(H):
                        assert res["cnt"][r, p, h] == len(D[r, h, p])
                        assert res["seg_off"][r, p, h] == cursor
                        if p != r:
                            vol += len(D[r, h, p])
                        if p != r or incl:
                            cursor += len(D[r, h, p])
                assert res["total"][r] == cursor
                assert res["volume"][r] == 2 * b * d * 2 * vol
                for h in range(H):
                    union = set().union(*[D[r, h, p] for p in range(P)])
                    assert _bits(res["U"][r, h], NB) == union


def test_direct_delivery_worked_example(oracle_mod):
    """Section 5.1: owner 0 holds A-D; consumers 1, 2, 3 need A, BC, D."""
    owner_blocks, needs, expect, expect_total = None, {}, None, None
    for line in open(os.path.join(GOLDEN, "direct_delivery_example.txt")):
        tok = line.split()
        if not tok or tok[0].startswith("#"):
            continue
        if tok[0] == "owner":
            owner_blocks = tok[3:]
        elif tok[0] == "consumer":
            needs[int(tok[1])] = tok[3:]
        elif tok[0] == "expect_from_owner0":
            expect = [int(t) for t in tok[1:]]
        elif tok[0] == "expect_total_from_owner0":
            expect_total = int(tok[1])
    P, per = 4, len(owner_blocks)
    NB = P * per
    rank = oracle_mod.placement_contiguous(NB, P)
    name_to_block = {n: idx for idx, n in enumerate(owner_blocks)}
    M = np.zeros((1, NB, NB), bool)
    for i in range(NB):
        M[0, i, i] = True  # every query block uses its own (local) KV block
    for c, names in needs.items():
        q_blocks = [i for i in range(NB) if rank[i] == c]
        for t, n in enumerate(names):
            M[0, q_blocks[t % len(q_blocks)], name_to_block[n]] = True
    res = oracle_mod.demand(_mask_from_bool(M), rank, P, 64, 64)
    assert [int(res["cnt"][c, 0, 0]) for c in (1, 2, 3)] == expect
    assert int(sum(res["cnt"][c, 0, 0] for c in (1, 2, 3))) == expect_total
    # nothing else crosses: every other remote count is zero
    for r in range(P):
        for p in range(1, P):
            if p != r:
                assert res["cnt"][r, p, 0] == 0


def test_band_mask_periodic_halo_closed_form(oracle_mod):
    """Section 4.3: every query at spatial position s attends [s-delta, s+delta] in each of T
    frames; under the interval-periodic layout an interior rank's remote demand is exactly
    2*delta*T blocks, an edge rank's delta*T."""
    T, B, G, delta, H, b = 5, 24, 4, 2, 2, 64
    NB = T * B
    M = np.zeros((H, NB, NB), bool)
    for t in range(T):
        for s in range(B):
            for t2 in range(T):
                for s2 in range(max(0, s - delta), min(B, s + delta + 1)):
                    M[:, t * B + s, t2 * B + s2] = True
    rank = oracle_mod.placement_periodic(NB, G, b, B * b, NB * b)
    assert list(rank[:B]) == [(G * s) // B for s in range(B)]
    assert np.all(rank.reshape(T, B) == rank[:B])
    res = oracle_mod.demand(_mask_from_bool(M), rank, G, b, 64)
    for r in range(G):
        remote = sum(int(res["cnt"][r, p, 0]) for p in range(G) if p != r)
        assert remote == (2 * delta * T if 0 < r < G - 1 else delta * T)
        assert res["volume"][r] == 2 * b * 64 * 2 * H * remote
    # the contiguous layout needs strictly more
    rank_c = oracle_mod.placement_contiguous(NB, G)
    res_c = oracle_mod.demand(_mask_from_bool(M), rank_c, G, b, 64)
    assert res_c["volume"].sum() > res["volume"].sum()


def test_all_ones_mask_and_single_rank(oracle_mod):
    H, NB, P, b, d = 2, 21, 4, 128, 64
    M = np.ones((H, NB, NB), bool)
    rank = oracle_mod.placement_contiguous(NB, P)
    res = oracle_mod.demand(_mask_from_bool(M), rank, P, b, d)
    own = [int((rank == p).sum()) for p in range(P)]
    for r in range(P):
        for p in range(P):
            assert np.all(res["cnt"][r, p] == own[p])
        assert res["volume"][r] == 2 * b * d * 2 * H * (NB - own[r])
    res1 = oracle_mod.demand(_mask_from_bool(M), np.zeros(NB, np.int32), 1, b, d)
    assert res1["volume"][0] == 0 and res1["total"][0] == 0


def test_two_ranks_ring_equals_direct(oracle_mod):
    """With two ranks a ring hop and a direct send are the same thing: the demanded set from the
    single peer is the whole remote demand."""
    rng = np.random.default_rng(5)
    H, NB = 2, 16
    M = rng.random((H, NB, NB)) < 0.2
    rank = oracle_mod.placement_contiguous(NB, 2)
    res = oracle_mod.demand(_mask_from_bool(M), rank, 2, 64, 64)
    for r in range(2):
        assert res["total"][r] == res["cnt"][r, 1 - r].sum()


def test_pack_equals_gather_by_enumerated_list(oracle_mod):
    rng = np.random.default_rng(7)
    H, b, d, P = 3, 64, 16, 3
    N = 5 * b + 23  # ragged last block
    NB = 6
    K = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    M = rng.random((H, NB, NB)) < 0.35
    M[:, :, NB - 1] |= rng.random((H, NB)) < 0.5  # make sure the ragged block is demanded
    rank = np.array([0, 1, 2, 0, 1, 2], np.int32)
    for incl in (False, True):
        res = oracle_mod.demand(_mask_from_bool(M), rank, P, b, d, include_local=incl)
        packed = oracle_mod.pack(K, V, res["U"], rank, b, P, res["total"], include_local=incl)
        D = _bruteforce_demand(M, rank, P)
        Kp = torch.zeros(H, NB * b, d, dtype=torch.bfloat16)
        Vp = torch.zeros(H, NB * b, d, dtype=torch.bfloat16)
        Kp[:, :N], Vp[:, :N] = K, V
        chunks = []
        for r in range(P):
            for p in range(P):
                if p == r and not incl:
                    continue
                for h in range(H):
                    for j in sorted(D[r, h, p]):
                        chunks.append(Kp[h, j * b:(j + 1) * b].reshape(-1))
                        chunks.append(Vp[h, j * b:(j + 1) * b].reshape(-1))
        expect = torch.cat(chunks).view(torch.int16).numpy().view(np.uint8) if chunks else np.zeros(0, np.uint8)
        assert packed.shape == expect.shape
        assert np.array_equal(packed, expect)
        assert int(res["total"].sum()) * 2 * b * d * 2 == packed.size


def test_pack_respects_destination_bases(oracle_mod):
    rng = np.random.default_rng(8)
    H, b, d, P, NB = 1, 64, 8, 2, 4
    N = NB * b
    K = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    M = np.ones((H, NB, NB), bool)
    rank = np.array([0, 0, 1, 1], np.int32)
    res = oracle_mod.demand(_mask_from_bool(M), rank, P, b, d)
    entry = 2 * b * d * 2
    dense = oracle_mod.pack(K, V, res["U"], rank, b, P, res["total"])
    base = np.array([3 * entry, 0], np.int64)  # swapped order with a gap
    moved = oracle_mod.pack(K, V, res["U"], rank, b, P, res["total"], dst_base=base)
    assert np.array_equal(moved[3 * entry:5 * entry], dense[:2 * entry])
    assert np.array_equal(moved[:2 * entry], dense[2 * entry:])
    assert not moved[2 * entry:3 * entry].any()


def test_placements(oracle_mod):
    assert list(oracle_mod.placement_contiguous(10, 4)) == [0, 0, 0, 1, 1, 2, 2, 2, 3, 3]
    # blocks aligned to frames: exactly floor(G*s/B)
    r = oracle_mod.placement_periodic(12, 3, 64, 6 * 64, 12 * 64)
    assert list(r) == [0, 0, 1, 1, 2, 2] * 2
    # text tail: round robin
    r = oracle_mod.placement_periodic(8, 2, 64, 3 * 64, 6 * 64)
    assert list(r[6:]) == [0, 1]


def test_consumer_view_rebuilds_exactly_the_demanded_blocks(oracle_mod):
    """Local blocks + the consumer's packed entries reproduce K/V on every block its rows keep, and
    nothing else is available (NaN) -- the packed layout and the locally derived offsets suffice."""
    rng = np.random.default_rng(11)
    H, b, d, P = 2, 64, 8, 3
    N = 5 * b + 30
    NB = 6
    K = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    V = torch.tensor(rng.standard_normal((H, N, d)), dtype=torch.float32).to(torch.bfloat16)
    M = rng.random((H, NB, NB)) < 0.4
    rank = np.array([0, 1, 2, 2, 0, 1], np.int32)
    dem = oracle_mod.demand(_mask_from_bool(M), rank, P, b, d)
    packed = oracle_mod.pack(K, V, dem["U"], rank, b, P, dem["total"])
    Kf = np.zeros((H, NB * b, d), np.float32)
    Kf[:, :N] = K.float().numpy()
    for r in range(P):
        Kr, Vr = oracle_mod.consumer_view(K, V, packed, dem, rank, b, r)
        for h in range(H):
            for j in range(NB):
                needed = rank[j] == r or any(M[h, i, j] for i in range(NB) if rank[i] == r)
                blk = Kr[h, j * b:(j + 1) * b]
                n_j = min(b, N - j * b)
                if needed:
                    assert np.array_equal(blk[:n_j], Kf[h, j * b:j * b + n_j])
                else:
                    assert np.isnan(blk).all()
