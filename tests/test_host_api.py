"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host helpers (geometry, top-k resolution, placements, argument validation) agree with the
oracle's independent definitions.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32197_b200 import build, binding as b
    build.build()
    b.lib()
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "sparsp.h")).read()
    declared = set(re.findall(r"SPARSP_API\s+[\w\s\*]+?\b(sparsp_\w+)\s*\(", header))
    assert declared and declared == set(binding.EXPORTS)
    L = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert getattr(L, name) is not None


def test_geometry_and_topk_resolution(binding, oracle_mod):
    from paper_2609_32197_b200 import synth
    for wl in synth.WORKLOADS.values():
        shape = binding.make_shape(wl.heads, wl.head_dim, wl.grid, wl.n_text, wl.block)
        g = binding.sparsp_geometry(shape)
        assert g.n_tokens == wl.n_tokens and g.n_blocks == wl.n_blocks
        assert g.n_words == (wl.n_blocks + 31) // 32
        flags = oracle_mod.text_block_flags(wl.n_video, wl.n_text, wl.block)
        assert g.n_video_blocks == int((flags == 0).sum()) == wl.nb_video
        for pct in (1, 5, 10, 15, 20, 25, 100):
            assert binding.sparsp_resolve_topk(pct, g.n_video_blocks) == oracle_mod.resolve_topk(pct, g.n_video_blocks)
    assert binding.sparsp_workspace_bytes(shape, 8) % 256 == 0


def test_placements_match_oracle(binding, oracle_mod):
    from paper_2609_32197_b200 import synth
    for wl in synth.WORKLOADS.values():
        shape = binding.make_shape(wl.heads, wl.head_dim, wl.grid, wl.n_text, wl.block)
        for P in (1, 2, 4, 8):
            assert np.array_equal(binding.sparsp_placement_contiguous(shape, P).numpy(),
                                  oracle_mod.placement_contiguous(wl.n_blocks, P))
            assert np.array_equal(binding.sparsp_placement_periodic(shape, P).numpy(),
                                  oracle_mod.placement_periodic(wl.n_blocks, P, wl.block, wl.frame_tokens, wl.n_video))


def test_host_side_argument_errors(binding):
    bad = binding.sparsp_shape(1, 2, 64, 0, 4, 4, 0, 64, 0, 0, 0)
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_geometry(bad)
    assert e.value.code == binding.SPARSP_ERR_INVALID_ARG and "non-positive" in str(e.value)
    big = binding.make_shape(1, 64, (100, 100, 100), 0, 64)  # 15625 blocks > 1024
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_geometry(big)
    assert e.value.code == binding.SPARSP_ERR_UNSUPPORTED
    ok = binding.make_shape(2, 64, (2, 8, 8), 0, 64)
    with pytest.raises(binding.SparspError):
        binding.sparsp_workspace_bytes(ok, 0)


def test_synthetic_inputs_are_seeded_and_shaped():
    import torch
    from paper_2609_32197_b200 import synth
    wl = synth.Workload("t", 2, 64, (2, 6, 8), 10, 64, 2, None, 2, seed=4)
    Q, K, V = synth.make_qkv(wl)
    Q2, K2, V2 = synth.make_qkv(wl)
    assert Q.shape == (2, 106, 64) and Q.dtype == torch.bfloat16
    assert torch.equal(Q, Q2) and torch.equal(K, K2) and torch.equal(V, V2)
    assert not torch.equal(Q[0], Q[1]) and not torch.equal(Q, K)
    # positional structure: a token's query is closer to its own key than to a far-away token's key
    q, k = Q.float(), K.float()
    assert (q[0, 5] * k[0, 5]).sum() > (q[0, 5] * k[0, 60]).sum()
    r = synth.shuffled_placement(37, 4, seed=1)
    assert torch.equal(r, synth.shuffled_placement(37, 4, seed=1))
    assert sorted(torch.bincount(r.long(), minlength=4).tolist()) == [9, 9, 9, 10]


def test_exchange_plan_matches_the_oracle(binding, oracle_mod):
    """sparsp_exchange_plan is host arithmetic: checked record by record against the oracle's transfer list,
    for several rank counts and chunkings, on demand counts the oracle computed from random masks."""
    import numpy as np
    import torch
    rng = np.random.default_rng(2)
    for (H, NB, P, steady, tail) in [(5, 40, 4, 1, 1), (8, 33, 3, 2, 4), (3, 20, 2, 2, 9), (6, 50, 7, 3, 2), (4, 12, 1, 1, 1)]:
        b, d = 64, 128
        M = rng.random((H, NB, NB)) < 0.1
        words = np.zeros((H, NB, (NB + 31) // 32), np.uint32)
        for h, i, j in zip(*np.nonzero(M)):
            words[h, i, j >> 5] |= np.uint32(1 << (int(j) & 31))
        rank = rng.integers(0, P, NB).astype(np.int32)
        dem = oracle_mod.demand(words, rank, P, b, d)
        want = oracle_mod.exchange_plan(dem["cnt"], dem["seg_off"], b, d, steady, tail)
        shape = binding.make_shape(H, d, (1, 1, NB * b), 0, b)
        got = binding.sparsp_exchange_plan(shape, P, torch.as_tensor(dem["cnt"])[None], torch.as_tensor(dem["seg_off"])[None],
                                           steady, tail)
        assert len(got) == len(want)
        for g, w in zip(got, want):
            assert g.batch == 0
            assert (g.consumer, g.producer, g.round, g.order, g.head_begin, g.head_end, g.entry_begin, g.n_entries,
                    g.byte_offset, g.n_bytes) == tuple(w[k] for k in (
                        "consumer", "producer", "round", "order", "head_begin", "head_end", "entry_begin",
                        "n_entries", "byte_offset", "n_bytes"))
    with pytest.raises(binding.SparspError):
        binding.sparsp_exchange_plan(shape, 1, torch.zeros(1, 1, 1, 4, dtype=torch.int32),
                                     torch.zeros(1, 1, 1, 4, dtype=torch.int64), 0, 1)
