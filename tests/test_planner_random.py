"""Randomised host-planner check (no GPU): for drawn shapes, placements with replicas,
TP pairs and block tables, replaying the exported segments with numpy copies must equal
the oracle on whole arenas, and the plan's byte counts must match the definitions."""
from __future__ import annotations

import dataclasses
import math

import numpy as np
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from helpers import FILL, rand_bytes
from test_planner import replay, run_oracle, oracle_sizes


@st.composite
def placements(draw, n_experts, max_ep=5):
    """A list of per-rank id lists in which every expert appears at least once, some
    twice (on different ranks), in a drawn slot order."""
    ep = draw(st.integers(1, max_ep))
    ranks = [[] for _ in range(ep)]
    for e in range(n_experts):
        home = draw(st.integers(0, ep - 1))
        ranks[home].append(e)
        if ep > 1 and draw(st.integers(0, 3)) == 0:
            other = draw(st.integers(0, ep - 2))
            other += other >= home
            ranks[other].append(e)
    return [draw(st.permutations(r)) for r in ranks]


@st.composite
def cases(draw):
    hkv = draw(st.sampled_from([1, 2, 4, 6, 8]))
    group = draw(st.sampled_from([1, 2, 3]))
    # TP degrees: divisors of Hkv, and multiples of it (more ranks than KV heads)
    divs = [t for t in (1, 2, 3, 4, 6, 8, 12, 16) if hkv % t == 0 or (t > hkv and t % hkv == 0)]
    c, d = draw(st.sampled_from(divs)), draw(st.sampled_from(divs))
    n_routed, n_shared = draw(st.integers(1, 7)), draw(st.integers(0, 2))
    sh = W.Shape(draw(st.integers(1, 3)), n_routed, n_shared, draw(st.sampled_from([3, 8, 16])),
                 draw(st.sampled_from([1, 5, 8])), math.lcm(hkv * group, c, d), hkv,
                 draw(st.sampled_from([1, 4, 8])),
                 draw(st.sampled_from([1, 3, 4])), draw(st.sampled_from([1, 2, 4])))
    B = sh.kv_block_tokens
    seq_lens = draw(st.lists(st.integers(0, 4 * B), min_size=0, max_size=4))
    used = sum(-(-n // B) for n in seq_lens)
    nb_old, nb_new = used + draw(st.integers(0, 3)), used + draw(st.integers(0, 3))
    seed = draw(st.integers(0, 2**31))
    order = draw(st.sampled_from(["random", "identity"]))
    if seq_lens and max(seq_lens) > 0:
        bo = W.make_block_table(W.rng.stream_key(seed, 1), seq_lens, B, nb_old)
        bn = W.make_block_table(W.rng.stream_key(seed, 2), seq_lens, B, nb_new, order=order)
    else:
        seq_lens, bo, bn = [], np.zeros((0, 0), np.int32), np.zeros((0, 0), np.int32)
    old = W.ParallelConfig(0, c, draw(placements(sh.n_experts)), max(nb_old, 1), seq_lens, bo)
    new = W.ParallelConfig(0, d, draw(placements(sh.n_experts)), max(nb_new, 1), seq_lens, bn)
    old.ep, new.ep = len(old.placement), len(new.placement)
    fused_w13 = draw(st.booleans())
    if not fused_w13:     # scale tensors travel with the plain [L][3][n][m] layout only
        sh = dataclasses.replace(sh, expert_scale_bytes=draw(st.sampled_from([0, 0, 4, 24, 48])))
    return W.Workload("drawn", sh, old, new, seed, fused_w13=fused_w13,
                      kv_head_major=draw(st.booleans()), fused_qkv=draw(st.booleans()))


@settings(max_examples=80, deadline=None, suppress_health_check=list(HealthCheck))
@given(cases())
def test_drawn_plans_replay_to_the_oracle(wl):
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_w13=wl.fused_w13,
                kv_head_major=wl.kv_head_major, fused_qkv=wl.fused_qkv) as plan:
        for phase in range(3):
            so, sn = oracle_sizes(wl, phase)
            assert plan.arena_bytes(phase, E.SIDE_OLD) == so
            assert plan.arena_bytes(phase, E.SIDE_NEW) == sn
            src = [rand_bytes((40 + phase, r), n) for r, n in enumerate(so)]
            want = [np.full(n, FILL, np.uint8) for n in sn]
            got = [np.full(n, FILL, np.uint8) for n in sn]
            run_oracle(wl, phase, src, want)
            segs = plan.segments(phase)
            replay(segs, src, got)
            for r in range(len(sn)):
                assert np.array_equal(got[r], want[r]), (phase, r)
            stt = plan.stats(phase)
            assert stt["bytes_moved"] == int((segs["run_bytes"] * segs["n_runs"]).sum())
            if phase == E.PHASE_EXPERTS and wl.shape.expert_scale_bytes:
                gaps = sum(oracle.expert_scale_base(wl.shape, len(p)) - wl.shape.n_layers * 3 * len(p)
                           * wl.shape.d_model * wl.shape.d_ff * wl.shape.elem_bytes for p in wl.new.placement)
                assert stt["bytes_moved"] == sum(sn) - gaps      # the gap before the scales is nobody's
            elif phase != E.PHASE_KV:
                assert stt["bytes_moved"] == sum(sn)
            else:
                sh = wl.shape
                used = sum(-(-n // sh.kv_block_tokens) for n in wl.old.seq_lens)
                heads = max(sh.n_kv_heads, wl.new.tp)    # replicas included
                assert stt["bytes_moved"] == (sh.n_layers * 2 * used * sh.kv_block_tokens
                                              * heads * sh.head_dim * sh.elem_bytes)


@st.composite
def inplace_cases(draw):
    """Slot tables with holes and replicas, a wanted set per new device that the free slots
    can hold (or, now and then, cannot)."""
    n_exp = draw(st.integers(1, 9))
    ep_old, ep_new = draw(st.integers(1, 4)), draw(st.integers(1, 5))
    old = []
    for r in range(ep_old):
        held = draw(st.lists(st.integers(0, n_exp - 1), unique=True, max_size=n_exp))
        table = list(held) + [-1] * draw(st.integers(0, 4))
        old.append(list(draw(st.permutations(table))))
    for e in range(n_exp):                      # every expert has a copy somewhere
        if not any(e in t for t in old):
            old[draw(st.integers(0, ep_old - 1))].append(e)
    want = [draw(st.lists(st.integers(0, n_exp - 1), unique=True, max_size=n_exp)) for _ in range(ep_new)]
    cap_new = [len(old[r]) if r < ep_old else len(want[r]) + draw(st.integers(0, 2)) for r in range(ep_new)]
    sh = W.Shape(draw(st.integers(1, 2)), n_exp, 0, draw(st.sampled_from([2, 8])), draw(st.sampled_from([1, 8])),
                 4, 4, 4, 4, draw(st.sampled_from([1, 2])))
    return sh, old, want, cap_new


@settings(max_examples=120, deadline=None, suppress_health_check=list(HealthCheck))
@given(inplace_cases())
def test_drawn_inplace_plans_replay_to_the_oracle(case):
    sh, old, want, cap_new = case
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    caps = [len(t) for t in old] + cap_new[len(old):]
    expect = [rand_bytes((60, r), sh.n_layers * 3 * c * m) for r, c in enumerate(caps)]
    got = [a.copy() for a in expect]
    try:
        new_slots = oracle.reshard_experts_inplace(sh, old, want, cap_new, expect)
    except ValueError as e:
        assert "free slots" in str(e)           # the only refusal these draws can produce
        try:
            E.InplacePlan(sh, old, want, cap_new, host_only=True)
        except E.EmoeError as err:
            assert err.code == 11
        else:
            raise AssertionError("the library accepted a step the capacity cannot hold")
        return
    with E.InplacePlan(sh, old, want, cap_new, host_only=True) as plan:
        assert plan.slot_tables() == new_slots
        snapshot = [a.copy() for a in got]
        for s in plan.segments(E.PHASE_EXPERTS):
            for i in range(int(s["n_runs"])):
                a = int(s["src_off"]) + i * int(s["src_pitch"])
                b = int(s["dst_off"]) + i * int(s["dst_pitch"])
                n = int(s["run_bytes"])
                got[int(s["dst_rank"])][b:b + n] = snapshot[int(s["src_rank"])][a:a + n]
        for r in range(len(expect)):
            assert np.array_equal(got[r], expect[r]), r
