"""The multi-GPU path of the benchmark is N replicas with their own batches and no data-path
collective; what the ranks share is the timing protocol (barrier, maximum over ranks, one line
from rank 0).  Covered here with two gloo ranks on CPU."""
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
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, w, l = bench.init_ranks("gloo")
    assert (r, w, l) == (rank, world, rank)
    dist.barrier()
    # each rank measured different times; the job reports the slowest
    mine = [1.0 + rank, 5.0 - rank, 0.25]
    got = bench.max_over_ranks(mine)
    # blocks are repeated until enough time has been measured: the ranks time differently (here one is twice as
    # fast) but must stop after the same block, since every block contains barriers
    calls = []

    def block(n):
        dist.barrier()
        calls.append(n)
        return 10.0 * (1 + rank)             # ms per call: rank 1 is the slow one
    med, n_blocks = bench.repeat_blocks(block, 5, min_s=0.25)
    out[rank] = (got, bench.rank_seed(rank), bench.job_throughput_gbs(w, 10 ** 9, got[0]), med, n_blocks, len(calls))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_the_slowest_time_and_draw_different_batches():
    world = 2
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (t0, s0, v0, m0, n0, c0), (t1, s1, v1, m1, n1, c1) = out[0], out[1]
    # 20 ms per call on the slow rank x 5 calls = 0.1 s per block: three blocks reach 0.25 s, on both ranks
    assert (m0, n0, c0) == (m1, n1, c1) == (20.0, 3, 3)
    assert t0 == t1 == [2.0, 5.0, 0.25]
    assert s0 != s1
    # 2 ranks x 1 GB over 2 ms
    assert abs(v0 - 1000.0) < 1e-9 and v0 == v1


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert bench.init_ranks("gloo") == (0, 1, 0)
    assert bench.max_over_ranks([3.0, 1.5]) == [3.0, 1.5]
    assert bench.repeat_blocks(lambda n: 100.0, 2, min_s=0.5) == (100.0, 3)
    assert not dist.is_initialized()
