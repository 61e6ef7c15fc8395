"""Multi-GPU is "replicas only" (the step has no exchange): the one piece of N>1 logic is how bench.py folds the
per-rank measurements into a whole-job number.  Checked here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, toks, e2e = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100 + rank, 7.0 * (rank + 1), dist, "cpu")
    out[rank] = (ms, toks, e2e)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_fold_max_time_and_summed_tokens():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank, args=(world, 29731, out), nprocs=world, join=True)
    for r in range(world):
        ms, toks, e2e = out[r]
        assert ms == 15.0 and toks == 201 and abs(e2e - 21.0) < 1e-9


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7, 2.0) == (3.5, 7, 2.0)
