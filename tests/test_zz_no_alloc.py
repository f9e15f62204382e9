"""emoe_reshard_kv_static: the KV re-split for callers that must not allocate device
memory - a serving process whose memory daemon already owns all of HBM, or a section
that cannot afford the implicit synchronisation of cudaMalloc.  Such a caller makes a
host-only plan (no CUDA call) and uses this entry point, whose only scratch is a fixed
array inside the library image.

The check: through the C ABI, on two calls in a row that share that array, the output
must be byte-identical to emoe_reshard_kv (the tolerance of every parity test here is
zero: this is byte movement).  Collected last on purpose (file name), and written so
that it passes alone in a fresh process as well as after the other tests."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest
import torch

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
        host_plan.reshard_kv_static(src, got)
        torch.cuda.synchronize()
        for r, (g, w) in enumerate(zip(got, want)):
            assert torch.equal(g, w), "%s: rank %d differs from emoe_reshard_kv" % (wl.name, r)
        # something was actually moved
        assert any(bool((w != WD.FILL_BYTE).any()) for w in want)


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
