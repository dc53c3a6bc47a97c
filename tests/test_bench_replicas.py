"""Multi-process plumbing of bench.py, on CPU with the gloo backend (world size 2): the job's
step time is the slowest rank's, the reported rate is the whole job's (replicas only: tokens are
independent, there is no collective on the data path), every rank draws its own inputs, and the
reference arm runs on rank 0 alone."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2503_15798_b200 import inputs

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 10.0 + 5.0 * rank  # rank 1 is the slow one
        ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
        value = bench.whole_job_tokens_per_s(world, 256, 100, ms)
        seeds = bench.rank_seeds(rank, layer=3, batch=5, m=64)
        ids = inputs.zipf_ids(64, 50304, seed=seeds["ids"])
        # every rank learns the others' id batches: replicas must not share them
        gathered = [torch.zeros(64, dtype=torch.int32) for _ in range(world)]
        dist.all_gather(gathered, torch.from_numpy(ids))
        out[rank] = {"ms": ms, "value": value, "seeds": seeds, "runs_reference": bench.reference_arm_runs_here(rank),
                     "distinct_batches": not torch.equal(gathered[0], gathered[1])}
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in res.values():
        assert r["ms"] == 15.0  # the max over ranks, on every rank
        assert np.isclose(r["value"], 2 * 256 * 100 / 15e-3)  # whole-job tokens/s, not per GPU
        assert r["distinct_batches"]
    assert res[0]["seeds"]["table"] != res[1]["seeds"]["table"] and res[0]["seeds"]["ids"] != res[1]["seeds"]["ids"]
    assert res[0]["seeds"]["router"] == res[1]["seeds"]["router"]  # same model on every replica
    assert res[0]["runs_reference"] and not res[1]["runs_reference"]


def test_single_process_needs_no_process_group():
    import bench

    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_tokens_per_s(1, 64, 10, 2.0) == 64 * 10 / 2e-3
