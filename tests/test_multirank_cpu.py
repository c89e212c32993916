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


def test_plain_gpus_flag_starts_one_rank_per_gpu():
    """`python bench.py --gpus N` without a launcher re-runs itself as N ranks on 127.0.0.1."""
    sys.path.insert(0, ROOT)
    import bench

    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "3"], port=29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "3"]
    # a port is found when none is given
    assert int(bench.spawn_command(2, [])[bench.spawn_command(2, []).index("--master-port") + 1]) > 0


# --------------------------------------------------------------------------- context-parallel decode plumbing
def _lse_merge_f64(o_parts, lse_parts):
    """The merge formula in float64 torch ops (stand-in for the CUDA merge kernel on CPU ranks)."""
    m = lse_parts.max(dim=0).values
    m_safe = torch.where(torch.isinf(m), torch.zeros_like(m), m)
    w = torch.exp(lse_parts - m_safe)
    wsum = w.sum(0)
    o = (w.unsqueeze(-1) * o_parts).sum(0) / torch.where(wsum > 0, wsum, torch.ones_like(wsum)).unsqueeze(-1)
    return o, m_safe + torch.log(wsum)


def _cp_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np

    from oracle import l4l_oracle as orc
    from paper_2608_21836_b200 import parallel

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, Hq, Hkv, D, L = 2, 4, 2, 8, 300
        g = torch.Generator().manual_seed(9)              # every rank builds the same full problem ...
        q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
        ck = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
        cv = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
        lens = [300, 130]
        # ... and keeps only its shard of every sequence's cache
        shard_len = []
        sk = torch.zeros(B, Hkv, L, D, dtype=torch.bfloat16)
        sv = torch.zeros(B, Hkv, L, D, dtype=torch.bfloat16)
        for b in range(B):
            t0, t1 = parallel.shard_bounds(lens[b], world, rank, granule=128)
            shard_len.append(t1 - t0)
            sk[b, :, :t1 - t0] = ck[b, :, t0:t1]
            sv[b, :, :t1 - t0] = cv[b, :, t0:t1]

        def local():
            o, lse = orc.decode(q, sk, sv, np.array(shard_len, np.int32), 0.3)
            return torch.from_numpy(o), torch.from_numpy(lse)

        o, lse = parallel.context_parallel_decode(local, _lse_merge_f64)
        want_o, want_lse = orc.decode(q, ck, cv, np.array(lens, np.int32), 0.3)
        out[rank] = (float(np.abs(o.numpy() - want_o).max()), float(np.abs(lse.numpy() - want_lse).max()), shard_len)
    finally:
        dist.destroy_process_group()


def test_context_parallel_decode_gathers_and_merges_over_two_gloo_ranks():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_cp_worker, args=(world, port, out), nprocs=world, join=True)
        for r in range(world):
            assert out[r][0] < 1e-12 and out[r][1] < 1e-12
        # the second sequence (130 tokens = 2 blocks of 128) gives rank 0 one block and rank 1 the ragged rest
        assert out[0][2] == [256, 128] and out[1][2] == [44, 2]


def test_shard_bounds_cover_the_sequence_once():
    sys.path.insert(0, ROOT)
    from paper_2608_21836_b200 import parallel

    for L in (0, 1, 127, 128, 129, 1000, 4096):
        for world in (1, 2, 3, 8):
            pieces = [parallel.shard_bounds(L, world, r) for r in range(world)]
            assert pieces[0][0] == 0 and pieces[-1][1] == L
            assert all(a[1] == b[0] for a, b in zip(pieces, pieces[1:]))
            assert all(t0 % 128 == 0 for t0, _ in pieces if t0 < L)
