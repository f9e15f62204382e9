"""GPU parity on drawn cases: shapes, placements with replicas, TP pairs and block tables
from the same strategy as the host-planner test, run through the CUDA kernels and
compared with the oracle byte for byte over whole arenas (deterministic draw)."""
from __future__ import annotations

import pytest
from hypothesis import HealthCheck, given, settings

import paper_2510_02613_b200 as E
from gpu_util import check_phase_full, check_step_full, make_plan
from test_planner_random import cases

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
