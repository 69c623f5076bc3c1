"""The N > 1 path of the benchmark on CPU: two gloo ranks agree on the slowest rank's time and
form the whole-job rate from it."""
import os
import socket

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2408_02897_b200 import ranks


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ranks.rank_info() == (rank, world, rank)
        ranks.barrier(world)
        my_ms = 10.0 + 5.0 * rank                    # rank 1 is the slow one
        slowest = ranks.max_over_ranks(my_ms, world)
        ranks.barrier(world)
        out.put((rank, slowest, ranks.whole_job_rate(3.0e12, world, slowest)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate in got:
        assert slowest == 15.0
        assert rate == pytest.approx(2 * 3.0e12 / 15.0e-3)


def test_single_process_needs_no_group():
    assert ranks.max_over_ranks(7.5, 1) == 7.5
    assert ranks.whole_job_rate(100.0, 1, 50.0) == pytest.approx(2000.0)
