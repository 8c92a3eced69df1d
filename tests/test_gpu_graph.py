"""The whole hot path (mask -> demand / pack -> attention) is stream-ordered work only: it can be captured in a
CUDA graph once and replayed, and a replay writes exactly the bytes that the plain calls write (which the parity
tests compare with the oracle; here the masks are compared with it once more, the rest bit for bit with the
plain calls).  No call may synchronise, allocate or read device data on the host."""
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


@pytest.mark.parametrize("d,b,n_text", [(64, 64, 0), (128, 128, 70), (128, 64, 33)])
def test_step_replayed_from_a_graph_equals_the_plain_calls(oracle_mod, binding, d, b, n_text):
    from paper_2609_32197_b200 import synth
    H, P, k = 3, 4, 6
    wl = synth.Workload("graph", H, d, (5, 12, 16), n_text, b, k, None, P, seed=17)
    Q, K, V = synth.make_qkv(wl, "cpu")
    shape = binding.make_shape(H, d, wl.grid, wl.n_text, b)
    g = binding.sparsp_geometry(shape)
    Qd, Kd, Vd = Q.cuda()[None].contiguous(), K.cuda()[None].contiguous(), V.cuda()[None].contiguous()
    ws = binding.make_workspace(shape, P)
    mo = binding.alloc_mask_outputs(shape, k, "cuda", with_list=True)
    do = binding.alloc_demand_outputs(shape, P)
    rank = torch.as_tensor(np.array([(j * 3 + j // 5) % P for j in range(g.n_blocks)], np.int32)).cuda()
    entry = 2 * b * d * 2
    cap = P * H * g.n_blocks * entry
    packed = torch.full((cap,), 0xAB, dtype=torch.uint8, device="cuda")
    O = torch.full_like(Qd, 3.0)
    lse = torch.full((1, H, g.n_tokens), 3.0, dtype=torch.float32, device="cuda")

    def step():
        binding.sparsp_block_mask(shape, Qd, Kd, k, mo["mask"], mo["kv_list"], mo["kv_count"], None, None, ws)
        binding.sparsp_demand_pack(shape, mo["mask"], rank, P, 0, Kd, Vd, do["union_mask"], do["cnt"], do["seg_offset"],
                                   do["seg_total"], do["volume_bytes"], packed, cap, None, ws)
        binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, mo["mask"], 0.0, O, lse, ws)

    step()
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    ref = oracle_mod.block_mask(Q, K, b, k, wl.n_text)
    assert np.array_equal(pu.u32(mo["mask"][0]), ref["mask"])
    outputs = (mo["mask"], mo["kv_list"], mo["kv_count"], do["union_mask"], do["cnt"], do["seg_offset"],
               do["seg_total"], do["volume_bytes"], packed, O, lse)
    plain = [t.clone() for t in outputs]

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    launches0 = binding.sparsp_launch_count()
    for rep in range(2):
        for t in outputs:   # a replay must rewrite every output
            t.fill_(0x5A if t.dtype == torch.uint8 else 5)
        graph.replay()
        torch.cuda.synchronize()
        assert binding.sparsp_status(ws) == binding.SPARSP_OK, binding.sparsp_last_error()
        for t, want in zip(outputs, plain):
            if t is packed:
                n = int(do["seg_total"].sum().item()) * entry
                assert torch.equal(t[:n], want[:n])
                assert bool((t[n:] == 0x5A).all())   # nothing past the planned bytes
            else:
                assert torch.equal(t.view(torch.uint8), want.view(torch.uint8)), rep
    assert binding.sparsp_launch_count() == launches0   # a replay goes through no library call
