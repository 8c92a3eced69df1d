"""GPU parity for the placement tools: permutation tables, token permutation (bytes, both directions, both
layouts), the sharing histogram; and the end-to-end property that attention commutes with the permutation."""
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


@pytest.mark.parametrize("d,b,layout", [(128, 128, "HND"), (64, 64, "NHD"), (128, 64, "NHD")])
def test_permutation_tables_and_token_permutation(oracle_mod, binding, d, b, layout):
    from paper_2609_32197_b200 import synth
    H, P = 3, 4
    wl = synth.Workload("perm", H, d, (3, 10, 17), 45, b, 3, None, P, seed=5)
    Q, _, _ = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b, layout=layout)
    for rank in (oracle_mod.placement_periodic(NB, P, b, wl.frame_tokens, wl.n_video),
                 synth.shuffled_placement(NB, P, seed=3).numpy()):
        bos, off, first = binding.sparsp_placement_permutation(shape, P, torch.as_tensor(rank))
        rb, ro, rf = oracle_mod.placement_permutation(rank, P, N, b)
        assert np.array_equal(bos.numpy(), rb) and np.array_equal(off.numpy(), ro) and np.array_equal(first.numpy(), rf)
        Xd = pu.to_layout(Q.cuda(), layout)
        Yd = torch.full_like(Xd, 7.0)
        binding.sparsp_permute_tokens(shape, Xd, Yd, bos.cuda(), off.cuda(), False)
        want = oracle_mod.permute_tokens(Q, rb, ro, b)
        assert torch.equal(pu.from_layout(Yd, layout).cpu(), want)
        Zd = torch.full_like(Xd, 7.0)
        binding.sparsp_permute_tokens(shape, Yd, Zd, bos.cuda(), off.cuda(), True)
        assert torch.equal(Zd, Xd)


def test_sharing_histogram_matches_the_oracle(oracle_mod, binding):
    from paper_2609_32197_b200 import synth
    H, P, d, b = 4, 4, 64, 64
    wl = synth.Workload("share", H, d, (4, 12, 16), 30, b, 7, None, P, seed=9)
    Q, K, V = synth.make_qkv(wl, "cpu")
    NB = wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    ws = binding.make_workspace(shape, P)
    mo = pu.gpu_block_mask(binding, shape, Q.cuda(), K.cuda(), wl.topk_abs, ws)
    mask_np = pu.u32(mo["mask"][0])
    for rank in (oracle_mod.placement_contiguous(NB, P), oracle_mod.placement_periodic(NB, P, b, wl.frame_tokens, wl.n_video)):
        hist = torch.full((1, P, 101), -1, dtype=torch.int64, device="cuda")
        binding.sparsp_sharing_histogram(shape, mo["mask"], torch.as_tensor(rank).cuda(), P, hist)
        want = oracle_mod.sharing_histogram(mask_np, rank, P)
        assert np.array_equal(hist[0].cpu().numpy(), want)
        assert want.sum() > 0


def test_attention_commutes_with_the_block_permutation(oracle_mod, binding):
    """Permuting Q, K, V by whole blocks, permuting the mask's rows and columns the same way, attending and
    permuting back gives the same output rows (the same key sets per query; only the order of the keys inside
    the softmax differs, hence a tolerance)."""
    from paper_2609_32197_b200 import synth
    H, P, d, b = 2, 3, 128, 128
    wl = synth.Workload("commute", H, d, (4, 16, 16), 0, b, 3, None, P, seed=13)   # 1024 tokens = 8 whole blocks
    Q, K, V = synth.make_qkv(wl, "cpu")
    N, NB = wl.n_tokens, wl.n_blocks
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    ws = binding.make_workspace(shape, P)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    mo = pu.gpu_block_mask(binding, shape, Qd, Kd, wl.topk_abs, ws)
    O = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mo["mask"], 0.0, O, None, ws)
    rank = synth.shuffled_placement(NB, P, seed=4)
    bos, off, _ = binding.sparsp_placement_permutation(shape, P, rank)
    bos_d, off_d = bos.cuda(), off.cuda()
    Qp, Kp, Vp = (torch.empty_like(x) for x in (Qd, Kd, Vd))
    for x, y in ((Qd, Qp), (Kd, Kp), (Vd, Vp)):
        binding.sparsp_permute_tokens(shape, x, y, bos_d, off_d, False)
    # mask in slot coordinates: M'[s, t] = M[block_of_slot[s], block_of_slot[t]]
    m = pu.u32(mo["mask"][0])
    Mb = np.zeros((H, NB, NB), bool)
    for j in range(NB):
        Mb[:, :, j] = (m[:, :, j >> 5] >> np.uint32(j & 31)) & 1
    Mp = Mb[:, bos.numpy()][:, :, bos.numpy()]
    words = np.zeros((1, H, NB, 1), np.uint32)
    for t in range(NB):
        words[0, :, :, 0] |= (Mp[:, :, t].astype(np.uint32) << np.uint32(t))
    Op = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qp, Kp, Vp, torch.as_tensor(words.view(np.int32)).cuda(), 0.0, Op, None, ws)
    back = torch.zeros_like(Qd)
    binding.sparsp_permute_tokens(shape, Op, back, bos_d, off_d, True)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    err = (back.float() - O.float()).abs()
    assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3


def test_placement_tools_reject_bad_arguments(binding):
    shape = binding.make_shape(2, 64, (2, 4, 16), 0, 64)      # two blocks
    with pytest.raises(RuntimeError):
        binding.sparsp_placement_permutation(shape, 2, torch.tensor([0, 5], dtype=torch.int32))
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(RuntimeError):
        binding.sparsp_permute_tokens(shape, z, z, z, z, False)       # same buffer
    with pytest.raises(RuntimeError):
        binding.sparsp_sharing_histogram(shape, z, z, 0, z)
