"""The multi-rank part of the benchmark (barrier, max of times, sum of units) on two gloo ranks on CPU."""

import os
import socket

import torch.multiprocessing as mp

from paper_2110_01595_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist_util.init("gloo")
    dist_util.barrier()
    t, u = dist_util.combine(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    out.put((rank, t, u))
    dist_util.barrier()
    dist_util.shutdown()


def test_combine_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results == [(0, 15.0, 300.0), (1, 15.0, 300.0)]


def test_combine_single_process_is_identity():
    assert dist_util.combine(3.5, 7.0) == (3.5, 7.0)
