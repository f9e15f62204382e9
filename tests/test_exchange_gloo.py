"""Control plane of the one-rank-per-process exchange on two gloo ranks (CPU): handle
table, which pointers each rank hands to the library, local-rank restriction, barriers.
The CUDA IPC calls and the plan are replaced by fakes; the data path is covered by the
GPU test."""
from __future__ import annotations

import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class FakeTensor:
    def __init__(self, ptr, n):
        self._p, self._n = ptr, n

    def data_ptr(self):
        return self._p

    def numel(self):
        return self._n


class FakePlan:
    """experts: 2 old ranks -> 2 new; attn / kv: 1 old rank -> 2 new."""
    OLD, NEW = (2, 1, 1), (2, 2, 2)

    def __init__(self):
        self.calls, self.local = [], []

    def num_ranks(self, phase, side):
        return (self.OLD, self.NEW)[side][phase]

    def set_local_rank(self, r):
        self.local.append(r)

    def _rec(self, name, src, dst, stream):
        self.calls.append((name, list(src), list(dst)))

    def reshard_experts(self, s, d, st=None):
        self._rec("experts", s, d, st)

    def reshard_attn(self, s, d, st=None):
        self._rec("attn", s, d, st)

    def reshard_kv(self, s, d, st=None):
        self._rec("kv", s, d, st)


class FakeStream:
    def synchronize(self):
        pass


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2510_02613_b200 import binding as B, exchange
        opened, closed = [], []
        # a handle encodes (owner rank, allocation id); mapping it yields a base unique to both
        B.ipc_export = lambda ptr: (("h%d" % (ptr // 1000)).encode(), ptr % 1000)
        B.ipc_open = lambda h: (opened.append(h), 500000 + 1000 * int(h[1:]))[1]
        B.ipc_close = lambda b: closed.append(b)
        plan = FakePlan()
        # rank r's old arenas live at 1000 * (10 r + phase) + 16
        own = lambda ph: FakeTensor(1000 * (10 * rank + ph) + 16, 64)
        old = [own(0), own(1) if rank == 0 else None, own(2) if rank == 0 else None]
        new = [FakeTensor(7000 + ph, 64) for ph in range(3)]
        exchange.exchange_step(dist, plan, rank, old, new, FakeStream())
        out.put((rank, plan.calls, plan.local, sorted(opened), sorted(closed)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_exchange_control_plane():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = {r[0]: r[1:] for r in (out.get(timeout=120) for _ in range(2))}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in (0, 1):
        calls, local, opened, closed = res[rank]
        assert local == [rank, -1]                       # restricted, then restored
        assert [c[0] for c in calls] == ["experts", "attn", "kv"]
        peer = 1 - rank
        # experts: own pointer for itself, the peer's allocation mapped at 500000 + 1000 * id, + offset 16
        src = calls[0][1]
        assert src[rank] == 1000 * (10 * rank) + 16
        assert src[peer] == 500000 + 1000 * (10 * peer) + 16
        # attn / kv: only rank 0 holds an old arena
        for ph in (1, 2):
            src = calls[ph][1]
            assert len(src) == 1
            assert src[0] == (1000 * ph + 16 if rank == 0 else 500000 + 1000 * ph + 16)
        # destinations: only this rank's entry is set
        for ph in range(3):
            dst = calls[ph][2]
            assert [d is not None for d in dst] == [r == rank for r in range(2)]
        # every mapping opened once and closed at the end
        assert len(opened) == len(set(opened)) == len(closed)
        assert len(opened) == (1 if rank == 0 else 3)
