"""The allocation-free planning call, for callers that may not allocate GPU memory (a plug-in inside
an application that owns all device memory, a loop that must stay out of the driver's allocator).

It has to return exactly what the regular planning call returns.  Two calls in a row are made on
purpose: the call keeps its scratch in an array inside the library that survives from call to call,
so the second call runs on top of the first one's leftovers (with a different placement and flag)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_noalloc_plan_matches_regular_plan_twice_in_a_row():
    from paper_2609_32197_b200 import binding, synth
    binding.lib()
    assert torch.cuda.is_available()
    wl = synth.Workload("noalloc", 3, 64, (5, 11, 13), 70, 64, 4, None, 4, seed=21)  # 785 tokens, 13 blocks
    Q, K, V = synth.make_qkv(wl, "cuda")
    shape = binding.make_shape(wl.heads, wl.head_dim, wl.grid, wl.n_text, wl.block)
    ws = binding.make_workspace(shape, 8)
    mo = binding.alloc_mask_outputs(shape, wl.topk_abs, with_list=False)
    binding.sparsp_block_mask(shape, Q, K, wl.topk_abs, mo["mask"], None, None, None, None, ws)
    NB = wl.n_blocks
    cases = [
        (4, 0, torch.tensor([(j * 5) % 4 for j in range(NB)], dtype=torch.int32)),
        (8, binding.SPARSP_INCLUDE_LOCAL, torch.tensor([(j * 3) % 8 for j in range(NB)], dtype=torch.int32)),
    ]
    for P, flags, rank in cases:
        rank_d = rank.cuda()
        ref = binding.alloc_demand_outputs(shape, P)
        binding.sparsp_demand_pack(shape, mo["mask"], rank_d, P, flags | binding.SPARSP_PLAN_ONLY, None, None,
                                   ref["union_mask"], ref["cnt"], ref["seg_offset"], ref["seg_total"],
                                   ref["volume_bytes"], None, 0, None, ws)
        got = binding.alloc_demand_outputs(shape, P)  # outputs are the caller's; the call allocates nothing
        for t in got.values():
            t.fill_(-7)
        binding.sparsp_demand_plan_noalloc(shape, mo["mask"], rank_d, P, flags, got["union_mask"], got["cnt"],
                                           got["seg_offset"], got["seg_total"], got["volume_bytes"])
        torch.cuda.synchronize()
        for name in ("union_mask", "cnt", "seg_offset", "seg_total", "volume_bytes"):
            assert torch.equal(got[name], ref[name]), (P, name)  # integer outputs: bit-exact
        assert int(got["volume_bytes"].sum()) > 0

    # sizes beyond the stated maximum are refused with a clear error, before anything is launched
    with pytest.raises(binding.SparspError) as e:
        binding.sparsp_demand_plan_noalloc(shape, mo["mask"], rank_d, 65, 0, got["union_mask"], got["cnt"],
                                           got["seg_offset"], got["seg_total"], got["volume_bytes"])
    assert e.value.code == binding.SPARSP_ERR_CAPACITY and "n_ranks <= 64" in str(e.value)
