"""One rank per process: the pull-based exchange (local-rank plans + CUDA IPC mappings of
the peers' old arenas), run as 2 and 4 processes that share cuda:0 with a gloo control
plane.  The processes' kernels never wait on one another (each pulls what it needs, a
barrier on the host separates the steps), so sharing one GPU is safe.  The union of what the
ranks wrote must equal the oracle's whole step byte for byte."""
from __future__ import annotations

import dataclasses
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads as W

pytestmark = pytest.mark.gpu
R = dataclasses.replace


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload(world: int):
    wl = W.make_workload("c1_tiny", n_layers=2)
    if world == 2:   # EP 2 -> 2 (round-robin -> contiguous ranges), TP 1 -> 2
        wl = R(wl, new=R(wl.new, ep=2, placement=W.place_contiguous(8, 2)))
    return wl        # world 4: EP 2 -> 4, TP 1 -> 2 as defined


def _worker(rank: int, world: int, port: int, out, force_bulk: bool = False, whole_step: bool = False):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import paper_2510_02613_b200 as E
        from paper_2510_02613_b200 import exchange
        from workloads import device as WD
        wl = _workload(world)
        kinds = (W.KIND_EXPERTS, W.KIND_ATTN, W.KIND_KV)
        with E.Plan(wl.shape, wl.old, wl.new) as plan:
            if force_bulk:      # TMA bulk copies reading the peers' mapped arenas
                plan.set_tuning(path=2)
            old, new = [], []
            for ph in range(3):
                so, sn = plan.arena_bytes(ph, E.SIDE_OLD), plan.arena_bytes(ph, E.SIDE_NEW)
                # this process owns rank index `rank` on either side, filled like the
                # single-process tests fill rank `rank`
                mine = None
                if rank < len(so):
                    mine = WD.alloc_filled(so, wl.seed, kinds[ph])[rank]
                old.append(mine)
                new.append(WD.alloc_const([sn[rank]])[0] if rank < len(sn) else None)
            torch.cuda.synchronize()
            exchange.exchange_step(dist, plan, rank, old, new, whole_step=whole_step)
            assert plan.device_status() == 0
            out.put((rank, [None if t is None else t.cpu().numpy() for t in new]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,force_bulk,whole_step", [(2, False, False), (4, False, False), (2, True, False),
                                                         (4, False, True), (2, True, True)])
def test_ranks_as_processes_pull_their_share(world, force_bulk, whole_step):
    import oracle
    from gpu_util import oracle_phase
    from workloads import device as WD
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out, force_bulk, whole_step)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    wl = _workload(world)
    kinds = (W.KIND_EXPERTS, W.KIND_ATTN, W.KIND_KV)
    sizes_old = [oracle.expert_arena_bytes(wl.shape, wl.old.placement),
                 oracle.attn_arena_bytes(wl.shape, wl.old.tp),
                 oracle.kv_arena_bytes(wl.shape, wl.old.tp, wl.old.kv_num_blocks)]
    sizes_new = [oracle.expert_arena_bytes(wl.shape, wl.new.placement),
                 oracle.attn_arena_bytes(wl.shape, wl.new.tp),
                 oracle.kv_arena_bytes(wl.shape, wl.new.tp, wl.new.kv_num_blocks)]
    for ph in range(3):
        src = [WD.host_slice(wl.seed, kinds[ph], r, 0, n) for r, n in enumerate(sizes_old[ph])]
        want = [np.full(n, WD.FILL_BYTE, np.uint8) for n in sizes_new[ph]]
        oracle_phase(wl, ph, src, want)
        for r, w in enumerate(want):
            assert np.array_equal(got[r][ph], w), "phase %d rank %d" % (ph, r)
