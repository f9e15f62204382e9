"""GPU parity on drawn cases: shapes, placements with replicas, TP pairs and block tables
from the same strategy as the host-planner test, run through the CUDA kernels and
compared with the oracle byte for byte over whole arenas (deterministic draw)."""
from __future__ import annotations

import pytest
from hypothesis import HealthCheck, given, settings

import paper_2510_02613_b200 as E
from gpu_util import check_phase_full, check_step_full, make_plan
from test_planner_random import cases, inplace_cases

pytestmark = pytest.mark.gpu


@settings(max_examples=40, deadline=None, derandomize=True, database=None,
          suppress_health_check=list(HealthCheck))
@given(cases())
def test_drawn_cases_match_the_oracle(wl):
    with make_plan(wl) as plan:
        for phase in range(3):
            check_phase_full(wl, plan, phase)
        for kv_mode in (2, 3, 4):
            plan.set_tuning(kv_mode=kv_mode, kv_order=2)
            check_phase_full(wl, plan, E.PHASE_KV)
        plan.set_tuning(path=2, max_ctas=2)
        for phase in range(3):
            check_phase_full(wl, plan, phase)
        check_step_full(wl, plan)
        plan.set_tuning()
        check_step_full(wl, plan)


@settings(max_examples=40, deadline=None, derandomize=True, database=None,
          suppress_health_check=list(HealthCheck))
@given(inplace_cases())
def test_drawn_inplace_steps_match_the_oracle(case):
    """The in-place expert step on drawn slot tables (holes, replicas, devices added and
    removed), default routing and forced onto the ring kernel; whole arenas against the oracle."""
    import numpy as np
    import torch
    import oracle
    import workloads as W
    from workloads import device as WD
    sh, old, want, cap_new = case
    try:
        plan = E.InplacePlan(sh, old, want, cap_new)
    except E.EmoeError as e:
        assert e.code == 11
        return
    with plan:
        for tuning in (dict(), dict(path=2, max_ctas=3)):
            plan.set_tuning(**tuning)
            dev = WD.alloc_filled(oracle.inplace_arena_bytes(sh, plan.caps), 31, W.KIND_EXPERTS)
            expect = [t.cpu().numpy() for t in dev]
            assert oracle.reshard_experts_inplace(sh, old, want, cap_new, expect) == plan.slot_tables()
            plan.reshard(dev)
            torch.cuda.synchronize()
            assert plan.device_status() == 0
            for r, (g, w) in enumerate(zip(dev, expect)):
                assert np.array_equal(g.cpu().numpy(), w), (tuning, r)
