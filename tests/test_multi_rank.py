"""The N > 1 path of the benchmark on CPU: two gloo ranks, each an independent replica.

The decode path has no exchange step, so ranks only meet at the barrier and at the
max-over-ranks of the timed region; this checks that plumbing and the whole-job figure."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 100.0 + 50.0 * rank                      # rank 1 is the slow replica
    dist.barrier()
    ms = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    out[rank] = (ms, bench.job_tokens_per_s(world, 64, 512, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    with mp.get_context("spawn").Manager() as mgr:      # never fork a process that already has threads
        out = mgr.dict()
        mp.spawn(_rank, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, rate = res[0]
    assert ms == 150.0
    assert rate == 2 * 64 * 512 / 0.150


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, None, torch.device("cpu")) == 12.5
    assert bench.job_tokens_per_s(1, 64, 512, 1000.0) == 64 * 512
