"""GPU parity for the CDF-threshold mask mode: masks and counts bit-exact against the oracle, and the
attention over such variable-length masks within tolerance."""
import numpy as np
import pytest
import torch

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32197_b200 import binding as b
    b.lib()
    return b


@pytest.mark.parametrize("d,b,layout", [(128, 128, "HND"), (64, 64, "NHD"), (128, 64, "HND"), (64, 128, "HND")])
@pytest.mark.parametrize("tau,scale", [(0.9, 0.0), (0.5, 0.0), (0.97, 2.5)])
def test_cdf_mask_matches_the_oracle_bit_for_bit(oracle_mod, binding, d, b, layout, tau, scale):
    from paper_2609_32197_b200 import synth
    H = 3
    wl = synth.Workload("cdf", H, d, (4, 13, 19), 100, b, 4, None, 2, seed=71)   # ragged video end, text tail
    Q, K, V = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    Qd, Kd, Vd = (pu.to_layout(x.cuda(), layout) for x in (Q, K, V))
    ws = binding.make_workspace(shape, 2)
    g = binding.sparsp_geometry(shape)
    mask = torch.zeros(1, H, NB, g.n_words, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, H, NB, dtype=torch.int32, device="cuda")
    binding.sparsp_block_mask_cdf(shape, Qd, Kd, tau, scale, mask, cnt, None, None, ws)
    torch.cuda.synchronize()
    ref = oracle_mod.block_mask_cdf(Q, K, b, tau, wl.n_text, scale)
    assert np.array_equal(pu.u32(mask[0]), ref["mask"])
    assert np.array_equal(cnt[0].cpu().numpy(), ref["kv_count"])
    assert ref["kv_count"].min() >= 1 and ref["kv_count"].max() > ref["kv_count"].min()   # rows differ in length
    # attention over the variable-length rows
    O = torch.zeros_like(Qd)
    lse = torch.zeros(1, H, N, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mask, 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(H) for i in range(0, NB, 3)] + [(0, NB - 1)]
    pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], b, pu.from_layout(O, layout), units, lse_gpu=lse[0])


def test_cdf_rejects_bad_arguments(binding):
    shape = binding.make_shape(2, 64, (2, 4, 8), 0, 64)
    ws = binding.make_workspace(shape, 2)
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    for tau, scale in [(0.0, 0.0), (1.5, 0.0), (float("nan"), 0.0), (0.9, -1.0)]:
        with pytest.raises(RuntimeError):
            binding.sparsp_block_mask_cdf(shape, z, z, tau, scale, z, None, None, None, ws)


@pytest.mark.parametrize("name,tau", [("mid", 0.9), ("cog", 0.85)])
def test_cdf_mask_full_size(oracle_mod, binding, name, tau):
    """Full-size workloads: CDF masks and counts compared in full; attention on a seeded sample of units."""
    from paper_2609_32197_b200 import synth
    wl = synth.WORKLOADS[name]
    H, d, b = wl.heads, wl.head_dim, wl.block
    Qd, Kd, Vd = synth.make_qkv(wl, "cuda")
    Q, K, V = Qd.cpu(), Kd.cpu(), Vd.cpu()
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    ws = binding.make_workspace(shape, wl.ranks)
    g = binding.sparsp_geometry(shape)
    mask = torch.zeros(1, H, NB, g.n_words, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, H, NB, dtype=torch.int32, device="cuda")
    binding.sparsp_block_mask_cdf(shape, Qd, Kd, tau, 0.0, mask, cnt, None, None, ws)
    torch.cuda.synchronize()
    ref = oracle_mod.block_mask_cdf(Q, K, b, tau, wl.n_text)
    gm = pu.u32(mask[0])
    assert np.array_equal(gm, ref["mask"]), f"mask differs on {(gm != ref['mask']).any(axis=2).sum()} rows"
    assert np.array_equal(cnt[0].cpu().numpy(), ref["kv_count"])
    O = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mask, 0.0, O, None, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    rng = np.random.default_rng(7)
    units = [(0, 0), (H - 1, NB - 1)] + [(int(rng.integers(H)), int(rng.integers(NB))) for _ in range(10)]
    pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], b, O, units)
    assert torch.isfinite(O.float()).all()


def test_cdf_mask_at_the_largest_block_count(oracle_mod, binding):
    """NB = 1000 (the limit is 1024): the kernel's per-row scratch is at its largest."""
    from paper_2609_32197_b200 import synth
    H, d, b = 1, 64, 64
    wl = synth.Workload("cdf_big", H, d, (10, 50, 128), 0, b, 4, None, 2, seed=3)   # 64000 tokens = 1000 blocks
    Q, K, V = synth.make_qkv(wl, "cpu")
    NB = wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    ws = binding.make_workspace(shape, 2)
    g = binding.sparsp_geometry(shape)
    mask = torch.zeros(1, H, NB, g.n_words, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, H, NB, dtype=torch.int32, device="cuda")
    binding.sparsp_block_mask_cdf(shape, Q.cuda(), K.cuda(), 0.9, 0.0, mask, cnt, None, None, ws)
    torch.cuda.synchronize()
    ref = oracle_mod.block_mask_cdf(Q, K, b, 0.9, 0)
    assert np.array_equal(pu.u32(mask[0]), ref["mask"])
    assert np.array_equal(cnt[0].cpu().numpy(), ref["kv_count"])


def test_cdf_rows_of_maximum_length(oracle_mod, binding):
    """1024 blocks (the largest supported row).  With all scores equal every term is the largest weight and every lane of
    the selection warp adds 32 of them (the 32-bit partial sums come closest to their range); one tie group, so every
    row keeps everything.  With random scores: masks and counts against the oracle, tau up to 1."""
    from paper_2609_32197_b200 import synth
    wl = synth.Workload("cdfmax", 1, 64, (16, 64, 64), 0, 64, 1, None, 2)
    assert wl.n_blocks == 1024
    shape = binding.make_shape(1, 64, wl.grid, 0, 64)
    ws = binding.make_workspace(shape, 2)
    g = binding.sparsp_geometry(shape)
    gen = torch.Generator().manual_seed(5)
    cases = [(torch.zeros(1, wl.n_tokens, 64), torch.ones(1, wl.n_tokens, 64), 0.5, True),
             (torch.randn(1, wl.n_tokens, 64, generator=gen) * 3, torch.randn(1, wl.n_tokens, 64, generator=gen), 0.9, False),
             (torch.randn(1, wl.n_tokens, 64, generator=gen) * 0.1, torch.randn(1, wl.n_tokens, 64, generator=gen), 1.0, False)]
    for Qf, Kf, tau, all_kept in cases:
        Q, K = Qf.to(torch.bfloat16), Kf.to(torch.bfloat16)
        mask = torch.zeros(1, 1, 1024, g.n_words, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, 1, 1024, dtype=torch.int32, device="cuda")
        binding.sparsp_block_mask_cdf(shape, Q.cuda()[None].contiguous(), K.cuda()[None].contiguous(), tau, 0.0, mask, cnt,
                                      None, None, ws)
        torch.cuda.synchronize()
        ref = oracle_mod.block_mask_cdf(Q, K, 64, tau, 0, 0.0)
        assert np.array_equal(pu.u32(mask[0]), ref["mask"])
        assert np.array_equal(cnt[0].cpu().numpy(), ref["kv_count"])
        if all_kept:
            assert int(ref["kv_count"].min()) == 1024
