"""The multi-GPU form of the benchmark is N independent replicas (the path has no exchange step): each rank
draws its own tokens, times its own steps, and the job's time is the maximum over ranks.  That host logic is
exercised here on CPU with two gloo ranks."""
import os
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from workloads import CONFIGS, make_streams
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        # rank 1 is the slower replica in the first figure, rank 0 in the second
        ms = bench.max_over_ranks([10.0 + 5.0 * rank, 7.0 - rank], world, device="cpu")
        s = make_streams(CONFIGS["C0"], bench.replica_seed(3, rank))
        out[rank] = (ms, float(s["y1"][0, 0]), bench.job_tokens_per_s(world, 64, 4, ms[0]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_draw_their_own_tokens():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == [15.0, 7.0] and res[1][0] == [15.0, 7.0]      # every rank sees the maximum
    assert res[0][1] != res[1][1]                                      # different tokens per replica
    assert np.isclose(res[0][2], 2 * 64 * 4 / 15e-3)                   # whole-job tokens/s over the slowest replica


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert bench.job_tokens_per_s(1, 8192, 10, 50.0) == 8192 * 10 / 0.05
