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
