"""The N>1 bookkeeping (replicas only: barrier, max-over-ranks time, summed throughput)
on two gloo ranks on the CPU."""
from __future__ import annotations

import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_02613_b200 import replicas


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        local_ms = 10.0 + 2.5 * rank            # rank 1 is the slow one
        job_ms = replicas.job_time_ms(local_ms, dist)
        out.put((rank, job_ms, replicas.job_throughput_gbs(1_000_000_000, world, job_ms)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_throughput():
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
    for rank, job_ms, gbs in got:
        assert job_ms == pytest.approx(12.5)             # max over ranks, on every rank
        assert gbs == pytest.approx(2 * 2 * 1e9 / 12.5e-3 / 1e9)   # 2 replicas x 2 x bytes / time


def test_single_process_is_the_identity():
    assert replicas.job_time_ms(3.25) == 3.25
    assert replicas.job_throughput_gbs(5 * 10**9, 1, 2.0) == pytest.approx(5000.0)
    with pytest.raises(ValueError):
        replicas.job_throughput_gbs(1, 1, 0.0)
