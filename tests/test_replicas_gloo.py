"""The N > 1 bookkeeping of the benchmark on CPU: two gloo ranks on 127.0.0.1.  Replicas share no data path; what has
to be right is that ranks take different inputs, that the reported time is the slowest rank's, and that the throughput
counts every rank's images."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

from paper_2507_19131_b200 import replicas  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        x = np.arange(2 * 5 * 3 * 4, dtype=np.float32).reshape(2, 5, 3, 4)
        mine = replicas.rank_input(x, rank)
        local_ms = 10.0 + 7.0 * rank                      # rank 1 is the slow one
        dist.barrier()
        worst = replicas.max_over_ranks(local_ms)
        gathered = [None] * world
        dist.all_gather_object(gathered, float(mine[0, 0, 0, 0]))
        out[rank] = (worst, replicas.job_throughput(1, 20, world, worst), gathered)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_whole_job():
    world, port = 2, _free_port()
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        worst, thr, firsts = out[rank]
        assert worst == 17.0                               # max over ranks, seen by every rank
        assert thr == pytest.approx(2 * 1 * 20 / 0.017)    # both ranks' images over the slowest rank's time
        assert firsts[0] != firsts[1]                      # the ranks work on different inputs


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(3.5) == 3.5
    x = np.arange(24, dtype=np.float32).reshape(1, 4, 3, 2)
    assert np.array_equal(replicas.rank_input(x, 0), x)
    assert np.array_equal(replicas.rank_input(x, 1)[0, 1], x[0, 0])
