"""A bounded device-side wait that runs out: the kernel records SPARSP_ERR_TIMEOUT with a `where` code in the
workspace's status words and returns normally; sparsp_status reports and resets it; the context and the
workspace stay usable.  The wait is provoked by the library's diagnostic call (a barrier nobody arrives on,
nothing else in flight), never by making a real kernel stall."""
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


def test_a_wait_that_runs_out_is_reported_and_the_next_call_succeeds(oracle_mod, binding):
    from paper_2609_32197_b200 import synth
    wl = synth.Workload("after_timeout", 2, 64, (2, 16, 16), 0, 64, 3, None, 2, seed=13)
    Q, K, V = synth.make_qkv(wl, "cpu")
    shape = binding.make_shape(2, 64, wl.grid, 0, 64)
    ws = binding.make_workspace(shape, 2)
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    binding.sparsp_selftest_wait_timeout(ws, 100_000)         # ~50 us of SM clocks
    assert binding.sparsp_status(ws) == binding.SPARSP_ERR_TIMEOUT
    text = binding.sparsp_last_error()
    assert "device status -5" in text and "detail 99 0 0" in text, text   # where = 99, CTA (0, 0)
    assert binding.sparsp_status(ws) == binding.SPARSP_OK     # reading reset it
    # the first report wins: a second timeout before the status is read does not overwrite the first
    binding.sparsp_selftest_wait_timeout(ws, 50_000)
    binding.sparsp_selftest_wait_timeout(ws, 50_000)
    assert binding.sparsp_status(ws) == binding.SPARSP_ERR_TIMEOUT
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    # ordinary calls on the same workspace and context still work and still match the oracle
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    ref, got = pu.check_mask(oracle_mod, binding, shape, Q, K, Qd, Kd, 3, 0, ws)
    O = torch.zeros_like(Qd)
    binding.sparsp_sparse_attn_fwd(shape, Qd, Kd, Vd, got["mask"], 0.0, O, None, ws)
    torch.cuda.synchronize()
    assert binding.sparsp_status(ws) == binding.SPARSP_OK
    units = [(h, i) for h in range(2) for i in range(wl.n_blocks)]
    pu.check_attn_units(oracle_mod, Q, K, V, ref["mask"], 64, O, units)


def test_selftest_rejects_bad_arguments(binding):
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for limit in (0, -5, 10**9):
        with pytest.raises(binding.SparspError) as e:
            binding.sparsp_selftest_wait_timeout(ws, limit)
        assert e.value.code == binding.SPARSP_ERR_INVALID_ARG
    with pytest.raises(binding.SparspError):
        binding.sparsp_selftest_wait_timeout(None, 1000)
