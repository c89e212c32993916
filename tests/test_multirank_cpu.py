"""The multi-GPU mode of bench.py runs independent replicas (the attention path has no exchange step);
what the ranks share is only the timing reduction. This covers it with two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r "measured" these times; the job's time is the slowest rank's
        mine = [10.0 + rank, 5.0 - rank, 1.0]
        got = bench.max_over_ranks(mine, world, "cpu")
        dist.barrier()
        out[rank] = got
    finally:
        dist.destroy_process_group()


def test_timings_are_reduced_with_max_over_two_gloo_ranks():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0, 1.0]


def test_whole_job_value_is_additive_over_replicas_and_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks([3.0, 4.0], 1) == [3.0, 4.0]
    one = bench.whole_job_value(1, 2.2e12, 2.0)
    assert abs(one - 1100.0) < 1e-9
    assert abs(bench.whole_job_value(8, 2.2e12, 2.0) - 8 * one) < 1e-9
