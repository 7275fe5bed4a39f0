"""Host-side logic of the multi-GPU benchmark path, on CPU with two `gloo` ranks: the path has no
data-path collective (ranks run independent replicas of the workload), so what has to be right is
that replicas differ, that the reported time is the maximum over ranks and that counts are summed."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2506_01084_b200 import synth_inputs as si
    times, counts = bench.reduce_over_ranks([10.0 + rank, 5.0 - rank], [100.0 * (rank + 1), 7.0], world,
                                            torch.device("cpu"))
    w = si.WORKLOADS["tiny"]
    toks = si.make_tokens(w, bench.replica_seed(rank))
    out[rank] = (times, counts, int(toks.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_rank_reduction_and_replica_seeds_with_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        times, counts, _ = res[rank]
        assert times == [11.0, 5.0]            # max over ranks of each time
        assert counts == [300.0, 14.0]         # sum over ranks of each count
    assert res[0][2] != res[1][2]              # the replicas consume different token streams


def test_single_rank_reduction_is_identity():
    import bench
    assert bench.reduce_over_ranks([1.5, 2.5], [3.0], 1, torch.device("cpu")) == ([1.5, 2.5], [3.0])
    assert bench.replica_seed(0) != bench.replica_seed(1)
