"""world_size-2 checks of the N > 1 plumbing on CPU (gloo): every rank runs its own replica, timings
reduce with MAX, work totals with SUM, and the whole-job value follows from those."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_32197_b200 import dist_util, synth
    wl = dist_util.replica_workload(synth.WORKLOADS["tiny"], rank)
    Q, _, _ = synth.make_qkv(wl, "cpu", heads=1)
    times, totals = dist_util.reduce_over_ranks({"step": 10.0 + 5 * rank, "attn": 7.0 - rank},
                                                {"flops": 1e9 * (rank + 1), "launches": 9})
    dist.barrier()
    out[rank] = (wl.seed, float(Q.float().sum()), times, totals)
    dist.destroy_process_group()


def test_two_ranks_replicas_and_reductions():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 0 and res[1][0] == 1            # each rank its own seed ...
    assert res[0][1] != res[1][1]                        # ... hence different inputs
    for r in range(world):
        times, totals = res[r][2], res[r][3]
        assert times == {"attn": 7.0, "step": 15.0}     # MAX over ranks
        assert totals == {"flops": 3e9, "launches": 18.0}  # SUM over ranks
    value = res[0][3]["flops"] / (res[0][2]["step"] * 1e-3)
    assert abs(value - 2e11) < 1


def test_single_process_passthrough():
    from paper_2609_32197_b200 import dist_util
    t, s = dist_util.reduce_over_ranks({"a": 1.5}, {"b": 2})
    assert t == {"a": 1.5} and s == {"b": 2}
