"""The multi-GPU benchmark's host logic on CPU: two gloo ranks, each with its own seeded batch and
its own measured time; the whole-job figure uses the slowest rank's time."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2602_12128_b200 import multi
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(multi.rank_seed(1000, rank))
    x = torch.randn(8, generator=g)
    ms = 2.0 + 3.0 * rank                       # rank 1 is the slow one
    slow = multi.max_over_ranks(ms, dist)
    gathered = [torch.zeros(8) for _ in range(world)]
    dist.all_gather(gathered, x)
    out.put((rank, slow, multi.whole_job_rate(100.0, world, slow), bool(torch.equal(gathered[0], gathered[1]))))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_max_time_and_distinct_batches():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, rate, same in res:
        assert slow == pytest.approx(5.0)
        assert rate == pytest.approx(2 * 100.0 / 5e-3)
        assert not same


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2602_12128_b200 import multi
    assert multi.max_over_ranks(3.5) == 3.5
    assert multi.whole_job_rate(10.0, 1, 1000.0) == 10.0
