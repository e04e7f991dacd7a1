"""The N > 1 path of the benchmark on CPU: two gloo ranks run the replica plumbing (barrier, maximum of the
per-rank device times, whole-job throughput) and must agree on the result."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_18145_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world_info(dist) == (rank, world)
        replicas.barrier(dist)
        # rank r "measured" 10 + r ms for the resident run and 20 - r ms end to end
        ms, ms_e2e = replicas.max_over_ranks([10.0 + rank, 20.0 - rank], dist)
        value = replicas.job_throughput(units_per_rank_per_step=16384, world=world, steps=5, ms_max=ms)
        out.put((rank, ms, ms_e2e, value))
        replicas.barrier(dist)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_aggregate_throughput():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, ms_e2e, value in res:
        assert ms == 11.0 and ms_e2e == 20.0                      # maxima over ranks, identical on both
        assert value == pytest.approx(16384 * 2 * 5 / 11.0e-3)   # all ranks' tokens over the slowest rank's time


def test_single_process_is_the_identity():
    assert replicas.world_info(None) == (0, 1)
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.job_throughput(100, 1, 2, 1000.0) == 200.0
    replicas.barrier(None)
