"""Randomised host-planner check (no GPU): for drawn shapes, placements with replicas,
TP pairs and block tables, replaying the exported segments with numpy copies must equal
the oracle on whole arenas, and the plan's byte counts must match the definitions."""
from __future__ import annotations

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
    return W.Workload("drawn", sh, old, new, seed, fused_w13=draw(st.booleans()),
                      kv_head_major=draw(st.booleans()))


@settings(max_examples=80, deadline=None, suppress_health_check=list(HealthCheck))
@given(cases())
def test_drawn_plans_replay_to_the_oracle(wl):
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_w13=wl.fused_w13,
                kv_head_major=wl.kv_head_major) as plan:
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
            if phase != E.PHASE_KV:
                assert stt["bytes_moved"] == sum(sn)
            else:
                sh = wl.shape
                used = sum(-(-n // sh.kv_block_tokens) for n in wl.old.seq_lens)
                heads = max(sh.n_kv_heads, wl.new.tp)    # replicas included
                assert stt["bytes_moved"] == (sh.n_layers * 2 * used * sh.kv_block_tokens
                                              * heads * sh.head_dim * sh.elem_bytes)
