"""emoe_reshard_kv_static: the KV re-split for callers that must not allocate device
memory - a serving process whose memory daemon already owns all of HBM, or a section
that cannot afford the implicit synchronisation of cudaMalloc.  Such a caller makes a
host-only plan (no CUDA call) and uses this entry point, whose only scratch is a fixed
array inside the library image.

The check: through the C ABI, on calls in a row that share that array, the output must
be byte-identical to emoe_reshard_kv AND to the CPU oracle (the tolerance of every
parity test here is zero: this is byte movement), and the calls must leave the amount
of free device memory unchanged.  Collected last on purpose (file name), and written
so that it passes alone in a fresh process as well as after the other tests."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from workloads import device as WD

pytestmark = pytest.mark.gpu


def _reference_and_static(wl):
    with E.Plan(wl.shape, wl.old, wl.new) as plan, \
            E.Plan(wl.shape, wl.old, wl.new, host_only=True) as host_plan:
        so = plan.arena_bytes(E.PHASE_KV, E.SIDE_OLD)
        sn = plan.arena_bytes(E.PHASE_KV, E.SIDE_NEW)
        src = WD.alloc_filled(so, wl.seed, W.KIND_KV)
        want = WD.alloc_const(sn)
        got = WD.alloc_const(sn)
        plan.reshard_kv(src, want)
        torch.cuda.synchronize()
        host_plan.reshard_kv_static(src, got)       # the first call on the device does the set-up
        torch.cuda.synchronize()
        for g in got:
            g.fill_(WD.FILL_BYTE)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        host_plan.reshard_kv_static(src, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
        expect = [np.full(n, WD.FILL_BYTE, np.uint8) for n in sn]
        oracle.reshard_kv(wl.shape, wl.old, wl.new, [t.cpu().numpy() for t in src], expect)
        for r, (g, w, x) in enumerate(zip(got, want, expect)):
            assert np.array_equal(g.cpu().numpy(), x), "%s: rank %d differs from the oracle" % (wl.name, r)
            assert torch.equal(g, w), "%s: rank %d differs from emoe_reshard_kv" % (wl.name, r)
        # something was actually moved
        assert any(bool((x != WD.FILL_BYTE).any()) for x in expect)


def test_static_entry_matches_reshard_kv_on_two_calls_in_a_row():
    # call 1: TP2 -> TP4 head re-split, 8192 block pairs fill part of the fixed array
    big = W.make_workload("c4_large", n_layers=1)
    _reference_and_static(big)
    # call 2: fewer pairs, other shape, TP unchanged; stale entries of call 1 stay behind
    small = W.make_workload("c1_tiny")
    small = dataclasses.replace(small, new=dataclasses.replace(small.new, tp=1))
    _reference_and_static(small)
    # call 3: the inverse direction of call 1 (TP4 -> TP2)
    _reference_and_static(big.swapped())
    # call 4: more TP ranks than KV heads (4 heads, TP2 -> TP8: every head on two new ranks)
    many = dataclasses.replace(big, new=dataclasses.replace(big.new, tp=8))
    _reference_and_static(many)


def test_static_entry_with_a_local_rank_writes_that_rank_only():
    """One rank per GPU: a plan restricted to new-rank index r writes only that rank's
    blocks; the other destination pointers may be NULL."""
    wl = W.make_workload("c4_large", n_layers=1)
    sizes_new = oracle.kv_arena_bytes(wl.shape, wl.new.tp, wl.new.kv_num_blocks)
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        src = WD.alloc_filled(plan.arena_bytes(E.PHASE_KV, E.SIDE_OLD), wl.seed, W.KIND_KV)
        expect = [np.full(n, WD.FILL_BYTE, np.uint8) for n in sizes_new]
        oracle.reshard_kv(wl.shape, wl.old, wl.new, [t.cpu().numpy() for t in src], expect)
        for r in (0, wl.new.tp - 1):
            plan.set_local_rank(r)
            mine = WD.alloc_const([sizes_new[r]])[0]
            plan.reshard_kv_static(src, [mine if k == r else None for k in range(wl.new.tp)])
            torch.cuda.synchronize()
            assert np.array_equal(mine.cpu().numpy(), expect[r]), "rank %d" % r


def test_static_entry_rejects_more_pairs_than_its_array_holds():
    B = 2
    n_blocks = 65536 + 1
    sh = W.Shape(1, 1, 0, 8, 8, 2, 2, 8, B, 2)
    bt = np.arange(n_blocks, dtype=np.int32)[None, :]
    cfg = W.ParallelConfig(1, 1, [[0]], n_blocks, [n_blocks * B], bt)
    new = dataclasses.replace(cfg, tp=2)
    with E.Plan(sh, cfg, new, host_only=True) as plan:
        src = [torch.zeros(16, dtype=torch.uint8, device="cuda")]
        dst = [torch.zeros(16, dtype=torch.uint8, device="cuda") for _ in range(2)]
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_kv_static(src, dst)
        assert ei.value.code == 11
        assert "capacity" in str(ei.value)
