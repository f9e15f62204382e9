"""One rank per GPU: the scale step as a pull-based exchange between processes.

Process g owns the old arenas of rank index g (where the old configuration has such a
rank) and the new arenas of rank index g.  Every process builds the same plan, restricts
it to its own destination rank (emoe_plan_set_local_rank) and pulls what it needs from its
peers' old arenas through CUDA IPC mappings: the library's kernels read a peer-mapped
pointer exactly as they read a local one (plain loads and per-CTA bulk copies).
torch.distributed carries the control plane only (handles, barriers); no collective
touches the data.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

from . import binding as B


class PeerArenas:
    """The old arenas of one phase as seen from this process: its own tensor (if it has
    one) and IPC mappings of the others'.  `opened` maps handle bytes to mapped bases and is
    shared by the phases of a step: arenas of one peer can lie in one allocation, and an
    allocation is mapped once per process."""

    def __init__(self, dist, rank: int, n_old_ranks: int, mine, opened: dict):
        world = dist.get_world_size()
        export = None
        if rank < n_old_ranks and mine is not None and mine.numel():
            export = B.ipc_export(mine.data_ptr())
        table = [None] * world
        dist.all_gather_object(table, export)        # control plane: 64-byte handles + offsets
        self.ptrs: List[Optional[int]] = []
        for r in range(n_old_ranks):
            if r == rank:
                self.ptrs.append(mine.data_ptr() if mine is not None and mine.numel() else None)
            elif r >= world or table[r] is None:
                self.ptrs.append(None)
            else:
                handle, offset = table[r]
                if handle not in opened:
                    opened[handle] = B.ipc_open(handle)
                self.ptrs.append(opened[handle] + offset)


class Exchange:
    """A prepared exchange: the plan restricted to this rank, the peers' old arenas mapped.
    Set-up and tear-down talk to the other processes (all of them must create and close
    their Exchange together); step() only enqueues this rank's kernels."""

    def __init__(self, dist, plan: "B.Plan", rank: int, old_arenas, new_arenas, whole_step: bool = False):
        """whole_step: run the three phases through ONE emoe_reshard_step call (its launch sets
        merged and side by side) instead of one call per phase."""
        self.dist, self.plan, self.rank = dist, plan, rank
        self.whole_step = whole_step
        self.opened: dict = {}
        self.calls = []
        self.step_src, self.step_dst = [], []
        plan.set_local_rank(rank)
        run = (plan.reshard_experts, plan.reshard_attn, plan.reshard_kv)
        try:
            for phase in range(3):
                n_old = plan.num_ranks(phase, B.SIDE_OLD)
                n_new = plan.num_ranks(phase, B.SIDE_NEW)
                pa = PeerArenas(dist, rank, n_old, old_arenas[phase], self.opened)
                lands = rank < n_new and new_arenas[phase] is not None
                dst = [new_arenas[phase] if (lands and r == rank) else None for r in range(n_new)]
                self.step_src.append(pa.ptrs)
                self.step_dst.append(dst)
                if lands:                            # else nothing of this phase lands here
                    self.calls.append((run[phase], pa.ptrs, dst))
        except Exception:
            self.close(barrier=False)
            raise

    def step(self, stream=None) -> None:
        """Enqueues this rank's share of the three phases on `stream`; no synchronisation."""
        if self.whole_step:
            if self.calls:
                self.plan.reshard_step(self.step_src, self.step_dst, stream)
            return
        for fn, src, dst in self.calls:
            fn(src, dst, stream)

    def bytes_pulled(self) -> dict:
        """Bytes this rank writes, and how many of them it reads from OTHER ranks' arenas."""
        total = remote = 0
        for phase in range(3):
            segs = self.plan.segments(phase)
            mine = segs[segs["dst_rank"] == self.rank]
            b = mine["run_bytes"].astype("int64") * mine["n_runs"].astype("int64")
            total += int(b.sum())
            remote += int(b[mine["src_rank"] != self.rank].sum())
        return dict(written=total, from_peers=remote)

    def close(self, barrier: bool = True) -> None:
        if barrier:
            self.dist.barrier()                      # nobody still reads a peer's old arena
        for base in self.opened.values():
            B.ipc_close(base)
        self.opened = {}
        self.calls = []
        self.plan.set_local_rank(-1)


def exchange_step(dist, plan: "B.Plan", rank: int, old_arenas, new_arenas, stream=None,
                  whole_step: bool = False) -> None:
    """Runs this rank's share of the three phases.

    old_arenas / new_arenas: per phase (experts, attn, kv) this process's own device tensor
    of rank index `rank`, or None where the configuration has no such rank.  All processes
    of `dist` must call this together.  Returns after this rank's kernels have finished and
    every rank has passed the closing barrier (peers may then free or reuse old arenas).
    """
    import torch

    dist.barrier()                                   # every old arena is complete
    ex = Exchange(dist, plan, rank, old_arenas, new_arenas, whole_step=whole_step)
    try:
        ex.step(stream)
        (stream.synchronize() if stream is not None else torch.cuda.synchronize())
    finally:
        ex.close()
