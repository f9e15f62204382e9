"""Placement chooser (host only): valid, balanced, and keeping as many experts in place as
the exhaustive search / the closed form say is possible."""
from __future__ import annotations

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from test_planner_random import placements


def check_valid(n_experts, new_p, ep_new):
    assert len(new_p) == ep_new
    assert sorted(e for p in new_p for e in p) == list(range(n_experts))      # every expert once
    sizes = [len(p) for p in new_p]
    assert max(sizes) - min(sizes) <= 1                                       # balanced
    assert all(p == sorted(p) for p in new_p)


def kept_count(old_p, new_p):
    return sum(1 for r, p in enumerate(new_p) if r < len(old_p) for e in p if e in old_p[r])


def closed_form_unreplicated(old_p, n_experts, ep_new):
    """Each expert held once: rank r keeps min(|P_old[r]|, cap_r); the E mod EP extra slots
    go to ranks that hold more than the base size."""
    base, extra = divmod(n_experts, ep_new)
    sizes = [len(p) for p in old_p[:ep_new]]
    return sum(min(s, base) for s in sizes) + min(extra, sum(1 for s in sizes if s > base))


def test_brute_force_equals_closed_form_on_unreplicated_cases():
    """Pins the exhaustive search itself: without replicas the optimum has a closed form."""
    for n, old_p, ep_new in [(6, W.place_contiguous(6, 2), 3), (7, W.place_contiguous(7, 3), 2),
                             (7, W.place_round_robin(7, 2), 4), (5, [[4, 0, 1, 2], [3]], 2),
                             (6, [[0, 1, 2, 3, 4, 5]], 3)]:
        assert oracle.max_kept_bruteforce(n, old_p, ep_new) == closed_form_unreplicated(old_p, n, ep_new)
    # hand-counted: experts {0,1} on rank 0, {1,2} on rank 1, EP stays 2, sizes 2 and 1:
    # rank 0 keeps 0 and 1, rank 1 keeps 2 -> all three stay
    assert oracle.max_kept_bruteforce(3, [[0, 1], [1, 2]], 2) == 3


@settings(max_examples=60, deadline=None)
@given(st.data())
def test_chooser_reaches_the_exhaustive_optimum(data):
    n = data.draw(st.integers(1, 7))
    old_p = data.draw(placements(n, max_ep=3))
    ep_new = data.draw(st.integers(1, 3))
    new_p, kept = E.place_min_transfer(n, old_p, ep_new)
    check_valid(n, new_p, ep_new)
    assert kept == kept_count(old_p, new_p)
    assert kept == oracle.max_kept_bruteforce(n, old_p, ep_new)


def test_paper_scenarios_and_bench_shapes():
    # EP4 -> EP6 with 12 experts: every old device keeps 2 of its 3 (contiguous ranges keep 3 in all)
    old_p = W.place_contiguous(12, 4)
    new_p, kept = E.place_min_transfer(12, old_p, 6)
    check_valid(12, new_p, 6)
    assert kept == 8 == closed_form_unreplicated(old_p, 12, 6)
    assert kept_count(old_p, W.place_contiguous(12, 6)) == 3
    # EP4 -> EP2: both remaining devices keep all they had
    new_p, kept = E.place_min_transfer(12, old_p, 2)
    assert kept == 6 and all(set(old_p[r]) <= set(new_p[r]) for r in range(2))
    # the mid-size and large shapes
    for n, a, b in [(60, 4, 6), (128, 3, 5), (64, 8, 12), (256, 16, 24)]:
        old_p = W.place_contiguous(n, a)
        new_p, kept = E.place_min_transfer(n, old_p, b)
        check_valid(n, new_p, b)
        assert kept == kept_count(old_p, new_p) == closed_form_unreplicated(old_p, n, b)
    # and it feeds the planner: fewer bytes to copy in the paged store
    sh = W.Shape(2, 60, 0, 64, 48, 4, 4, 16, 4, 2)
    old_p = W.place_contiguous(60, 4)
    chosen, _ = E.place_min_transfer(60, old_p, 6)
    a = E.vmm_dry_run(sh, old_p, W.place_contiguous(60, 6), 1 << 21)
    b = E.vmm_dry_run(sh, old_p, chosen, 1 << 21)
    assert a["slabs_copied"] == 45 * 6 and b["slabs_copied"] == 20 * 6
    assert b["slabs_remapped"] == 40 * 6 and a["slabs_remapped"] == 15 * 6


def test_chooser_rejects_bad_input():
    with pytest.raises(E.EmoeError) as ei:
        E.place_min_transfer(4, [[0, 1], [2]], 2)          # expert 3 held by nobody
    assert ei.value.code == 3
    with pytest.raises(E.EmoeError) as ei:
        E.place_min_transfer(4, [[0, 1], [2, 3]], 65)
    assert ei.value.code == 9
