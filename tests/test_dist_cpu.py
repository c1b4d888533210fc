"""The N > 1 path of the benchmark on CPU: two gloo ranks, max-over-ranks time, summed work."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2011_05630_b200 import dist as D


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is slower: the job runs at the slowest rank's pace, the work adds up
    value, ms = D.job_throughput(local_ms_total=10.0 * (rank + 1), local_units=320.0)
    out.put((rank, value, ms, D.shard_batch(33, rank, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms, shard in got:
        assert ms == 20.0 and value == pytest.approx(640.0 / 0.020)
    assert got[0][3] == (0, 17) and got[1][3] == (17, 33)


def test_single_process_needs_no_process_group():
    value, ms = D.job_throughput(4.0, 32.0)
    assert ms == 4.0 and value == pytest.approx(8000.0)
    assert [D.shard_batch(10, r, 4) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]
