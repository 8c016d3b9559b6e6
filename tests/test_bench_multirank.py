"""The N > 1 path of bench.py is replicas only: no data-path collective, just the whole-job reduction
(slowest rank's time, summed work).  Exercised here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, world, 0)
        ms = 10.0 if rank == 0 else 12.5                     # rank 1 is the slow one
        tokens = 1000 if rank == 0 else 1100                 # replicas draw different documents
        results[rank] = bench.whole_job(ms, tokens, steps=5, world=world, device="cpu")
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_whole_job_reduction_over_two_gloo_ranks():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_rank_main, args=(world, port, results), nprocs=world, join=True)
        for rank in range(world):
            ms_max, tokens_all, value = results[rank]
            assert ms_max == 12.5 and tokens_all == 2100.0
            assert abs(value - 2100.0 * 5 / 12.5e-3) < 1e-6


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job(4.0, 92868, 10, 1, "cpu") == (4.0, 92868.0, 92868.0 * 10 / 4.0e-3)
