"""In-place expert step (emoe_plan_create_inplace): host planner against the oracle on CPU,
kernels against the oracle on the GPU.  Arenas are capacity-strided, only arrivals move."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from helpers import rand_bytes

CASES = {
    "grow_2_3": ([[0, 1, 2, -1, -1], [3, 4, 5, -1, -1]], [[0, 1], [3, 4], [2, 5]], [5, 5, 3]),
    "grow_with_swaps": ([[0, 1, 2, -1, -1, -1], [3, 4, 5, -1, -1, -1]],
                        [[5, 0, 4], [1, 3], [2, 0, 3]], [6, 6, 4]),
    "shrink_3_2": ([[0, 1, -1, -1], [2, 3, -1, -1], [4, 5, -1]], [[0, 1, 4, 2], [3, 5, 2]], [4, 4]),
    "holes_first": ([[-1, 0, -1, 1], [-1, -1, 2, 3]], [[3, 2, 0], [1, 3]], [4, 4]),
    "replicated": ([[0, 1, -1, -1], [1, 2, -1, -1]], [[0, 2, 1], [0, 1], [1, 2, 0]], [4, 4, 3]),
    "nothing_moves": ([[0, 1, -1], [2, -1, 3]], [[1, 0], [3, 2]], [3, 3]),
    "consecutive_arrivals": ([[0, 1, 2, 3, 4, 5], [-1] * 8], [[0, 1, 2, 3, 4, 5], [1, 2, 3, 4, 0]], [6, 8]),
}


def shape_for(old, d_model=8, d_ff=6, n_layers=2, elem_bytes=2):
    n_exp = 1 + max(e for t in old for e in t)
    return W.Shape(n_layers, n_exp, 0, d_model, d_ff, 8, 4, 4, 4, elem_bytes)


def arenas_for(sh, old, cap_new, key):
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    caps = [len(t) for t in old] + list(cap_new)[len(old):]
    return [rand_bytes((key, r), sh.n_layers * 3 * c * m) for r, c in enumerate(caps)]


@pytest.mark.parametrize("name", sorted(CASES))
def test_inplace_plan_replayed_on_the_host_equals_the_oracle(name):
    old, want, cap_new = CASES[name]
    sh = shape_for(old)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    with E.InplacePlan(sh, old, want, cap_new, host_only=True) as plan:
        assert plan.slot_tables() == oracle.inplace_slots(old, want, cap_new)
        expect = arenas_for(sh, old, cap_new, 5)
        got = [a.copy() for a in expect]
        oracle.reshard_experts_inplace(sh, old, want, cap_new, expect)
        n_dev = max(len(old), len(want))
        assert plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_OLD) == [a.size for a in got[:len(old)]]
        assert plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_NEW) == [a.size for a in got[:len(want)]]
        segs = plan.segments(E.PHASE_EXPERTS)
        snapshot = [a.copy() for a in got]          # sources are read as they were before the step
        for s in segs:
            for i in range(int(s["n_runs"])):
                a = int(s["src_off"]) + i * int(s["src_pitch"])
                b = int(s["dst_off"]) + i * int(s["dst_pitch"])
                n = int(s["run_bytes"])
                got[int(s["dst_rank"])][b:b + n] = snapshot[int(s["src_rank"])][a:a + n]
        for r in range(n_dev):
            assert np.array_equal(got[r], expect[r]), "device %d" % r
        arrivals = sum(1 for r, t in enumerate(plan.slot_tables()) for s_, e in enumerate(t)
                       if e >= 0 and not (r < len(old) and old[r][s_] == e))
        st = plan.stats(E.PHASE_EXPERTS)
        assert st["bytes_moved"] == arrivals * sh.n_layers * 3 * m
        assert st["bytes_read"] <= st["bytes_moved"]


def test_consecutive_arrivals_from_consecutive_slots_are_one_segment():
    old, want, cap_new = CASES["consecutive_arrivals"]
    with E.InplacePlan(shape_for(old), old, want, cap_new, host_only=True) as plan:
        segs = plan.segments(E.PHASE_EXPERTS)
        m = 8 * 6 * 2
        # arrivals 1,2,3,4 come from slots 1..4 of device 0 into slots 0..3: one 4-matrix run;
        # arrival 0 (slot 4) comes from slot 0
        assert sorted(int(s["run_bytes"]) for s in segs) == [m, 4 * m]


def test_inplace_validation_codes():
    sh = W.Shape(1, 4, 0, 8, 8, 8, 4, 4, 4, 2)
    def code(old, want, cap):
        with pytest.raises(E.EmoeError) as ei:
            E.InplacePlan(sh, old, want, cap, host_only=True)
        return ei.value.code
    assert code([[0, 1, -1]], [[2, 3]], [3]) == 3            # 2 and 3 have no copy anywhere
    assert code([[0, 1, 2, 3]], [[0], [1, 2, 3]], [4, 2]) == 11   # new device too small
    assert code([[0, 1, 2, -1], [3, -1]], [[0, 1, 2], [3, 0, 1]], [4, 2]) == 11   # one free slot, two arrivals
    assert code([[0, 1, 2, 3]], [[0, 1, 2, 3]], [5]) == 1    # a staying device cannot change capacity
    assert code([[0, 0, 1, 2, 3]], [[0]], [5]) == 3          # an expert twice in one table
    assert code([[0, 1, 2, 3]], [[0, 0]], [4]) == 3          # wanted twice
    assert code([[0, 1, 2, 9]], [[0]], [4]) == 3             # id out of range
    with E.InplacePlan(sh, [[0, 1, 2, 3]], [[0, 1], [2, 3]], [4, 2], host_only=True) as plan:
        with pytest.raises(E.EmoeError) as ei:               # not an out-of-place plan
            plan.reshard_experts([0], [0, 0])
        assert ei.value.code == 1
        with pytest.raises(E.EmoeError) as ei:               # host-only
            plan.reshard([0, 0])
        assert ei.value.code == 8


# ---- GPU --------------------------------------------------------------------------------

def _gpu_case(sh, old, want, cap_new, tuning=None, seed=7):
    import torch
    from workloads import device as WD
    with E.InplacePlan(sh, old, want, cap_new) as plan:
        if tuning:
            plan.set_tuning(**tuning)
        sizes = oracle.inplace_arena_bytes(sh, plan.caps)
        dev = WD.alloc_filled(sizes, seed, W.KIND_EXPERTS)
        expect = [t.cpu().numpy() for t in dev]
        new_slots = oracle.reshard_experts_inplace(sh, old, want, cap_new, expect)
        assert plan.slot_tables() == new_slots
        plan.reshard(dev)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        for r, (g, w) in enumerate(zip(dev, expect)):
            g = g.cpu().numpy()
            if not np.array_equal(g, w):
                bad = np.flatnonzero(g != w)
                raise AssertionError("device %d: %d bytes differ, first at %d" % (r, bad.size, bad[0]))
        return dev, new_slots


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(CASES))
@pytest.mark.parametrize("tuning", [None, dict(path=1), dict(path=2, max_ctas=5)],
                         ids=["default", "vector", "ring"])
def test_gpu_inplace_small_cases(name, tuning):
    old, want, cap_new = CASES[name]
    _gpu_case(shape_for(old, d_model=64, d_ff=96, n_layers=3), old, want, cap_new, tuning)


def _slots_with_spare(placement, want):
    """Old slot tables with exactly as many spare slots as the step needs arrivals."""
    old = []
    for r, p in enumerate(placement):
        arrivals = len([e for e in want[r] if e not in p]) if r < len(want) else 0
        old.append(list(p) + [-1] * arrivals)
    return old


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["c2_mid", "c3_fine", "c4_large"])
def test_gpu_inplace_full_width_layers(name):
    """Two full-width layers of the benchmark shapes, contiguous-range placements and the
    placement that keeps the most experts in place; whole arenas against the oracle."""
    import dataclasses
    wl = W.make_workload(name, n_layers=2)
    n_exp = wl.shape.n_experts
    for want in (wl.new.placement, E.place_min_transfer(n_exp, wl.old.placement, wl.new.ep)[0]
                 if name != "c3_fine" else wl.new.placement[::-1][:wl.new.ep]):
        want = [list(p) for p in want]
        old = _slots_with_spare(wl.old.placement, want)
        cap_new = [len(t) for t in old] + [len(want[r]) + 1 for r in range(len(old), len(want))]
        cap_new = cap_new[:len(want)]
        _gpu_case(wl.shape, old, want, cap_new, seed=wl.seed)


@pytest.mark.gpu
def test_gpu_inplace_chain_of_steps_up_and_down():
    """2 -> 4 -> 6 -> 4 -> 2 devices, every placement chosen from the previous one; the same
    arenas are carried from step to step, slots freed by one step are reused by the next."""
    import torch
    from workloads import device as WD
    sh = W.Shape(2, 24, 0, 64, 96, 8, 8, 16, 4, 2)
    cap = 16
    placement = W.place_contiguous(24, 2)
    slots = [list(p) + [-1] * (cap - len(p)) for p in placement]
    sizes = oracle.inplace_arena_bytes(sh, [cap] * 6)
    dev = WD.alloc_filled(sizes, 99, W.KIND_EXPERTS)
    host = [t.cpu().numpy() for t in dev]
    for ep_new in (4, 6, 4, 2):
        held = [[e for e in t if e >= 0] for t in slots]
        want, _ = E.place_min_transfer(24, held, ep_new)
        n_dev = max(len(slots), ep_new)
        with E.InplacePlan(sh, slots, want, [cap] * ep_new) as plan:
            plan.reshard(dev[:n_dev])
            torch.cuda.synchronize()
            new_slots = oracle.reshard_experts_inplace(sh, slots, want, [cap] * ep_new, host[:n_dev])
            assert plan.slot_tables() == new_slots
        for r in range(n_dev):
            assert np.array_equal(dev[r].cpu().numpy(), host[r]), (ep_new, r)
        slots = new_slots
