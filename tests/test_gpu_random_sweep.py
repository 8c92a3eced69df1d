"""Seeded random sweep of the whole path against the oracle: head dim, block size, head count, rank count, grid, text
length, layout, k, placement and input statistics are all drawn per case.  Three kinds of case: the generator's
structured inputs; unstructured inputs with per-token norm profiles (log-normal, up to e^1.5 spread: stress for the
norm bounds and the frozen reference of the attention kernel); and the same with an ARBITRARY mask handed to the
demand / pack / attention calls (random density per row, some rows empty, some full), which the selection step never
produces but the calls must handle.  Integers and bytes bit-exact, attention within the stated tolerance on every row."""
import numpy as np
import pytest
import torch

import parity_util as pu

pytestmark = pytest.mark.gpu

N_CASES = 60


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32197_b200 import binding as b
    b.lib()
    assert torch.cuda.is_available()
    return b


def _draw(rng):
    from paper_2609_32197_b200 import synth
    while True:
        d, b = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
        H, P = int(rng.integers(1, 4)), int(rng.integers(1, 9))
        grid = (int(rng.integers(1, 9)), int(rng.integers(4, 28)), int(rng.integers(4, 30)))
        n_text = int(rng.choice([0, 0, int(rng.integers(1, 300))]))
        wl = synth.Workload("sweep", H, d, grid, n_text, b, 1, None, P, seed=int(rng.integers(0, 1 << 30)))
        if wl.nb_video >= 1:
            return wl


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_case(oracle_mod, binding, case):
    from paper_2609_32197_b200 import synth
    rng = np.random.default_rng(9000 + case)
    wl = _draw(rng)
    H, d, b, P, N, NB = wl.heads, wl.head_dim, wl.block, wl.ranks, wl.n_tokens, wl.n_blocks
    layout = str(rng.choice(["HND", "NHD"]))
    k = int(rng.integers(1, wl.nb_video + 1))
    kind = case % 3
    if kind == 0:
        Q, K, V = synth.make_qkv(wl, "cpu")
    else:
        g = torch.Generator().manual_seed(int(rng.integers(0, 1 << 30)))
        sq = torch.exp(torch.randn(H, N, 1, generator=g) * float(rng.choice([0.0, 0.5, 1.5])))
        sk = torch.exp(torch.randn(H, N, 1, generator=g) * float(rng.choice([0.0, 0.5, 1.5])))
        Q = (torch.randn(H, N, d, generator=g) * sq * float(rng.choice([0.3, 1.0, 3.0]))).to(torch.bfloat16)
        K = (torch.randn(H, N, d, generator=g) * sk).to(torch.bfloat16)
        V = (torch.randn(H, N, d, generator=g) * float(rng.choice([0.5, 1.0, 2.0]))).to(torch.bfloat16)
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    Qd, Kd, Vd = (pu.to_layout(x.cuda(), layout) for x in (Q, K, V))
    ws = binding.make_workspace(shape, P)

    # step 1: pooled vectors, mask, kept lists, counts -- bit-exact
    ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Qd, Kd, k, wl.n_text, ws)
    mask_np, mask_d = ref["mask"], got["mask"]
    if kind == 2:
        Wd = mask_np.shape[2]
        dens = rng.random((H, NB, 1)) ** 2
        dens[rng.random((H, NB, 1)) < 0.1] = 0.0
        dens[rng.random((H, NB, 1)) < 0.05] = 1.0
        bits = rng.random((H, NB, Wd * 32)) < dens
        bits[:, :, NB:] = False
        mask_np = np.packbits(bits.reshape(H, NB, Wd, 32), axis=3, bitorder="little").view(np.uint32).reshape(H, NB, Wd)
        mask_d = torch.as_tensor(mask_np.view(np.int32)).cuda()[None].contiguous()

    # step 2: unions, counts, offsets, volumes and packed bytes for a random placement -- bit-exact
    rank_np = rng.integers(0, P, NB).astype(np.int32)
    rank_d = torch.as_tensor(rank_np).cuda()
    dg = pu.gpu_demand_pack(binding, shape, mask_d, rank_d, P, 0, Kd, Vd, ws)
    assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
    dref = pu.check_demand(oracle_mod, binding, shape, mask_np, rank_np, P, False, dg)
    packed_ref = oracle_mod.pack(K, V, dref["U"], rank_np, b, P, dref["total"])
    assert np.array_equal(dg["packed"].cpu().numpy()[:packed_ref.size], packed_ref)
    assert bool((dg["packed"][packed_ref.size:] == 0xAB).all())

    # step 3: every row of the output and of the log-sum-exp
    O = torch.full_like(Qd, 7.0)
    lse = torch.full((1, H, N), 7.0, dtype=torch.float32, device="cuda")
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mask_d, 0.0, O, lse, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
    o_ref, lse_ref = oracle_mod.attn_all(Q, K, V, mask_np, b)
    o_got = pu.from_layout(O, layout).float().cpu().numpy()
    assert np.isfinite(o_got).all()
    err = np.abs(o_got - o_ref)
    # the stated tolerance holds for |O| < 4 (half a bf16 unit of the output is 2^-7 there, 2^-6 for 4 <= |O| < 8, ...);
    # cases drawn with 2 sigma V may exceed that, and the tolerance grows with the output's own rounding
    grow = max(1.0, float(np.abs(o_ref).max()) / 4.0)
    assert err.max() <= pu.ATTN_MAX_ABS * grow and err.mean() <= pu.ATTN_MEAN_ABS * grow, (err.max(), err.mean(), grow)
    l_got = lse[0].cpu().numpy()
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isfinite(l_got), fin)          # rows without a kept key: -inf on both sides
    assert bool((o_got[~fin] == 0).all())                   # ... and an all-zero output row
    if fin.any():
        # an fp32 result: 2e-2, or a few units in the last place where extreme norms push the value into the thousands
        tol = 2e-2 + 8 * np.spacing(np.abs(lse_ref[fin]).astype(np.float32))
        assert bool((np.abs(l_got[fin] - lse_ref[fin]) <= tol).all())
