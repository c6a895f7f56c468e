"""The benchmark's multi-rank plumbing on CPU: two gloo processes, barrier, max over ranks."""
import os
import socket

import torch.multiprocessing as mp

from paper_2608_15522_b200 import dist_timing as dt


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, size, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(size), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist = dt.init("gloo")
    assert dist is not None and dt.world() == (rank, rank, size)
    dt.barrier(dist)
    # rank r pretends its step took 10 + 5 r ms and its end-to-end step 20 - r ms
    got = dt.max_over_ranks(dist, [10.0 + 5.0 * rank, 20.0 - rank])
    out.put((rank, got))
    dt.barrier(dist)
    dist.destroy_process_group()


def test_two_ranks_take_the_max_over_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [15.0, 20.0]
    # whole-job rate: both ranks did the same units; the slowest rank's time counts
    assert dt.whole_job_rate(3.0, 2, 15.0) == 3.0 * 2 / 0.015


def test_single_process_defaults():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert dt.world() == (0, 0, 1)
    assert dt.init("gloo") is None
    assert dt.max_over_ranks(None, [1.5, 2.5]) == [1.5, 2.5]
    dt.barrier(None)
