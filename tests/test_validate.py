"""The host-side bounds and race check of copy plans (emoe_segments_validate /
emoe_plan_validate): plans made by the library pass; segment lists with a run shifted out
of its arena, onto a neighbour's bytes or away from the bytes it should cover are caught."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest

import paper_2510_02613_b200 as E
import workloads as W
from test_planner import small

R = dataclasses.replace


@pytest.mark.parametrize("name", ["c1_tiny", "c2_mid", "c3_fine", "c4_large"])
def test_library_plans_pass_their_own_check(name):
    wl = small(name)
    variants = [dict(), dict(fused_w13=True, kv_head_major=True), dict(fused_qkv=True), dict(attn_replicas=3)]
    for kw in variants:
        for w in (wl, wl.swapped()):
            with E.Plan(w.shape, w.old, w.new, host_only=True, **kw) as plan:
                plan.validate()
    scaled = R(wl, shape=R(wl.shape, elem_bytes=1, expert_scale_bytes=24))
    with E.Plan(scaled.shape, scaled.old, scaled.new, host_only=True) as plan:
        plan.validate()
    with E.InplacePlan(W.Shape(2, 6, 0, 8, 8, 4, 4, 4, 4, 2), [[0, 1, 2, -1, -1], [3, 4, 5, -1]],
                       [[0, 3], [4, 1, 5], [2]], [5, 4, 2], host_only=True) as plan:
        plan.validate()


def test_corrupted_segment_lists_are_caught():
    wl = small("c4_large")
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        for phase, tile in ((E.PHASE_EXPERTS, True), (E.PHASE_ATTN, True), (E.PHASE_KV, False)):
            segs = plan.segments(phase)
            ao, an = plan.arena_bytes(phase, E.SIDE_OLD), plan.arena_bytes(phase, E.SIDE_NEW)
            assert E.segments_validate(segs, ao, an, tile) == -1
            k = len(segs) // 2
            bad = segs.copy(); bad["dst_off"][k] += 16                     # onto a neighbour / out of the arena
            if tile:          # (in a KV pool the neighbour may be an unmapped block: nothing to collide with)
                assert E.segments_validate(bad, ao, an, tile) != -1
            bad = segs.copy(); bad["dst_off"][k] = bad["dst_off"][k - 1]; bad["dst_rank"][k] = bad["dst_rank"][k - 1]
            assert E.segments_validate(bad, ao, an, tile) != -1            # onto another segment's bytes
            bad = segs.copy(); bad["src_off"][k] = ao[int(bad["src_rank"][k])]   # source run past the arena's end
            assert E.segments_validate(bad, ao, an, tile) == k
            bad = segs.copy(); bad["dst_rank"][k] = len(an)                # rank out of range
            assert E.segments_validate(bad, ao, an, tile) == k
            bad = segs.copy(); bad["dst_pitch"][k] = 2**62                 # would overflow a naive bound check
            if int(bad["n_runs"][k]) > 1:
                assert E.segments_validate(bad, ao, an, tile) == k
            if tile:                                                       # a dropped segment leaves a hole
                assert E.segments_validate(np.delete(segs, k), ao, an, True) != -1
                assert E.segments_validate(np.delete(segs, k), ao, an, False) == -1
            dup = np.concatenate([segs, segs[k:k + 1]])                    # two writers of the same bytes
            assert E.segments_validate(dup, ao, an, False) != -1
    assert E.strerror(12).startswith("a copy run")
