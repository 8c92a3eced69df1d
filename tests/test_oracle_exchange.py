"""Pins for the oracle's transfer list of the demand-routed exchange (Sections 5.1, 5.2, 7.1, 7.2): the
paper's direct-delivery example, the round structure as permutations, byte ranges that tile each
consumer's buffer exactly, chunk order."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


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


def _random_case(oracle_mod, seed, H=5, NB=40, P=4, dens=0.08):
    rng = np.random.default_rng(seed)
    M = rng.random((H, NB, NB)) < dens
    rank = rng.integers(0, P, NB).astype(np.int32)
    dem = oracle_mod.demand(_mask_words(M), rank, P, 64, 32)
    return M, rank, dem


def test_direct_delivery_example_by_rounds(oracle_mod):
    """Section 5.1: owner 0 holds A-D; ranks 1, 2, 3 need A, BC, D.  Rank 0 serves ring distance 1, 2, 3 in
    rounds 0, 1, 2 with 1, 2, 1 blocks and nothing else crosses."""
    expect = None
    for line in open(os.path.join(GOLDEN, "direct_delivery_example.txt")):
        tok = line.split()
        if tok and tok[0] == "expect_from_owner0":
            expect = [int(t) for t in tok[1:]]
    P, per = 4, 4
    NB = P * per
    rank = oracle_mod.placement_contiguous(NB, P)
    M = np.zeros((1, NB, NB), bool)
    for i in range(NB):
        M[0, i, i] = True
    needs = {1: [0], 2: [1, 2], 3: [3]}
    for c, blocks in needs.items():
        for j in blocks:
            M[0, c * per, j] = True
    dem = oracle_mod.demand(_mask_words(M), rank, P, 64, 64)
    plan = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], 64, 64)
    from0 = {t["round"]: (t["consumer"], t["n_entries"]) for t in plan if t["producer"] == 0}
    assert [from0[k] for k in range(3)] == [(1, expect[0]), (2, expect[1]), (3, expect[2])]
    assert sum(t["n_entries"] for t in plan if t["producer"] != 0) == 0
    assert sum(t["n_bytes"] for t in plan) == sum(expect) * 2 * 64 * 64 * 2


def test_every_round_is_a_permutation_and_every_pair_meets_once(oracle_mod):
    for P in (2, 3, 4, 7):
        _, _, dem = _random_case(oracle_mod, P, P=P)
        plan = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], 64, 32)
        seen = set()
        for k in range(P - 1):
            hop = [(t["consumer"], t["producer"]) for t in plan if t["round"] == k]
            assert sorted(c for c, _ in hop) == list(range(P))       # everyone receives once ...
            assert sorted(p for _, p in hop) == list(range(P))       # ... and sends once
            assert all((c - p) % P == k + 1 for c, p in hop)          # ring distance k + 1
            seen.update(hop)
        assert seen == {(c, p) for c in range(P) for p in range(P) if c != p}
        assert all(t["round"] < P - 1 for t in plan)


def test_byte_ranges_tile_each_consumer_buffer(oracle_mod):
    """The ranges of a consumer's transfers are disjoint, cover its buffer exactly, add up to its exchange
    volume, and each is the run of its (producer, heads) in pack order -- for any chunking."""
    b, d = 64, 32
    entry = 2 * b * d * 2
    for seed, steady, tail in [(1, 1, 1), (2, 2, 5), (3, 3, 2), (4, 8, 8)]:
        _, _, dem = _random_case(oracle_mod, seed)
        P, _, H = dem["cnt"].shape
        plan = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], b, d, steady, tail)
        for r in range(P):
            mine = [t for t in plan if t["consumer"] == r]
            spans = sorted((t["byte_offset"], t["byte_offset"] + t["n_bytes"]) for t in mine if t["n_bytes"])
            assert all(a1 == b0 for (_, a1), (b0, _) in zip(spans, spans[1:]))
            assert (spans[0][0] if spans else 0) == 0
            assert (spans[-1][1] if spans else 0) == int(dem["total"][r]) * entry == int(dem["volume"][r])
            for t in mine:
                p, h0, h1 = t["producer"], t["head_begin"], t["head_end"]
                assert t["entry_begin"] == int(dem["seg_off"][r, p, h0])
                assert t["n_entries"] == int(dem["cnt"][r, p, h0:h1].sum())
            for k in range(P - 1):
                hop = [t for t in mine if t["round"] == k]
                want = min(H, tail if k == P - 2 else steady)
                assert len(hop) == want
                assert sorted((t["head_begin"], t["head_end"]) for t in hop) == \
                    [((c * H) // want, ((c + 1) * H) // want) for c in range(want)]


def test_sparsest_chunk_goes_last(oracle_mod):
    _, _, dem = _random_case(oracle_mod, 9, H=8, dens=0.12)
    plan = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], 64, 32, 4, 4)
    P = dem["cnt"].shape[0]
    for r in range(P):
        for k in range(P - 1):
            hop = sorted((t for t in plan if t["consumer"] == r and t["round"] == k), key=lambda t: t["order"])
            sizes = [t["n_entries"] for t in hop]
            assert sizes == sorted(sizes, reverse=True)
            assert sizes[-1] == min(sizes)
            for a, c in zip(hop, hop[1:]):
                assert a["n_entries"] > c["n_entries"] or a["head_begin"] < c["head_begin"]


def test_plan_lists_exactly_the_demanded_blocks(oracle_mod):
    """Brute force: the (head, block) pairs a transfer stands for, enumerated from the mask, are the entries
    [entry_begin, entry_begin + n_entries) of the consumer's packed order."""
    M, rank, dem = _random_case(oracle_mod, 11, H=3, NB=24, P=3, dens=0.15)
    H, NB, _ = M.shape
    P = 3
    plan = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], 64, 32, 2, 3)
    for r in range(P):
        order = [(p, h, j) for p in range(P) if p != r for h in range(H) for j in range(NB)
                 if rank[j] == p and any(M[h, i, j] for i in range(NB) if rank[i] == r)]
        for t in (t for t in plan if t["consumer"] == r):
            got = order[t["entry_begin"]:t["entry_begin"] + t["n_entries"]]
            want = [(t["producer"], h, j) for h in range(t["head_begin"], t["head_end"]) for j in range(NB)
                    if rank[j] == t["producer"] and any(M[h, i, j] for i in range(NB) if rank[i] == r)]
            assert got == want
