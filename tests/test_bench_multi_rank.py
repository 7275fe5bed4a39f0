"""Host-side logic of the multi-GPU benchmark path, on CPU with two `gloo` ranks: the path has no
data-path collective (ranks run independent replicas of the workload), so what has to be right is
that replicas differ, that the reported time is the maximum over ranks and that counts are summed."""
import json
import os
import subprocess
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


def test_gpus_flag_starts_the_ranks_itself():
    # `bench.py --gpus 2` without a launcher's environment must start two ranks, rendezvous on
    # 127.0.0.1, reduce over them and print one line from rank 0.  --stub replaces the GPU work by
    # fixed per-rank numbers (rank r: 10 + r ms, 1000 (r + 1) tokens) so this runs on CPU with gloo.
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub"], env=env,
                       stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["stub"] is True
    assert line["ms_per_step"] == 11.0                       # max over ranks
    assert abs(line["value"] - 3000.0 / 0.011) < 1e-6        # summed tokens / max time
    assert line["config"]["replica_seeds"] == [1000, 1001]


def test_region_planning():
    import bench
    assert bench.plan_regions(20, 0.25, 10 ** 6) == 66       # 1.1 x 0.3 s / (20 x 0.25 ms)
    assert bench.plan_regions(20, 0.25, 100) == 5            # bounded by the codebook room in steps
    assert bench.plan_regions(256, 2.0, 10 ** 6) == 1        # one region already covers 0.3 s
    assert bench.plan_regions(20, 0.25, -5) == 1


def test_inputs_shared_between_workloads_equal_fresh_draws():
    # bench.Inputs keeps generated tensors per (shape, seed) and, for a workload that differs from a
    # cached one only in the merge size, draws the position table alone: the result must be what
    # synth_inputs.make_encoder draws for that workload from scratch
    import bench
    from paper_2506_01084_b200 import synth_inputs as si
    base = si.Workload("w3", V=300, d=64, dtype="bf16", B=2, T=32, M=3, cap=16, zipf_s=1.1, copy_p=0.3,
                       seg_min=2, seg_max=5, steps=1, enc_layers=2, enc_heads=2, enc_dff=128)
    other = base.scaled(name="w5", M=5)
    inp = bench.Inputs(torch.device("cpu"))
    first = inp.encoder(base, 77)
    again = inp.encoder(other, 77)
    fresh = si.make_encoder(other, 77)
    assert len(again) == len(fresh) and again[0].shape == (5, 64)
    for a, b in zip(again, fresh):
        assert torch.equal(a, b)
    for a, b in zip(first, si.make_encoder(base, 77)):
        assert torch.equal(a, b)
    assert inp.encoder(base, 77)[3] is first[3]                # cached, not drawn again
    te, tu = inp.tables(base, 5)
    fe, fu = si.make_tables(base, 5)
    assert torch.equal(te, fe) and torch.equal(tu, fu)
    assert inp.to_dev(te) is inp.to_dev(te)
