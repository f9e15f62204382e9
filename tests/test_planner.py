"""Host planner (no GPU): replaying the exported segment list with plain numpy
copies must reproduce the oracle byte for byte; destination runs must tile the
planned destination set exactly once; bad inputs map to the documented codes."""
from __future__ import annotations

import ctypes
import dataclasses
import re
import os

import numpy as np
import pytest

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from helpers import FILL, rand_bytes

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def small(name):
    """Per-layer structure of the named workload with tiny matrices."""
    wl = W.make_workload(name)
    sh = wl.shape
    L = 2
    if name == "c1_tiny":
        sh = dataclasses.replace(sh, n_layers=L, d_model=32, d_ff=16)
    else:
        sh = dataclasses.replace(sh, n_layers=L, d_model=16, d_ff=8, head_dim=8)
        # keep the block-table structure but only the first sequences
        def cut(cfg, pool):
            sl = list(cfg.seq_lens[:2])
            bt = cfg.block_table[:2].copy()
            return dataclasses.replace(cfg, seq_lens=sl, block_table=bt)
        wl = dataclasses.replace(wl, old=cut(wl.old, 0), new=cut(wl.new, 0))
    return dataclasses.replace(wl, shape=sh)


def replay(segs, src, dst):
    for s in segs:
        for i in range(int(s["n_runs"])):
            a = int(s["src_off"]) + i * int(s["src_pitch"])
            b = int(s["dst_off"]) + i * int(s["dst_pitch"])
            n = int(s["run_bytes"])
            dst[int(s["dst_rank"])][b:b + n] = src[int(s["src_rank"])][a:a + n]


def arenas(sizes, key):
    return [rand_bytes((key, r), n) for r, n in enumerate(sizes)]


def run_oracle(wl, phase, src, dst):
    if phase == E.PHASE_EXPERTS:
        oracle.reshard_experts(wl.shape, wl.old.placement, wl.new.placement, src, dst,
                               fused_w13=wl.fused_w13)
    elif phase == E.PHASE_ATTN:
        oracle.reshard_attn(wl.shape, wl.old.tp, wl.new.tp, src, dst, fused_qkv=wl.fused_qkv,
                            replicas=wl.attn_replicas)
    else:
        oracle.reshard_kv(wl.shape, wl.old, wl.new, src, dst, head_major=wl.kv_head_major)


def oracle_sizes(wl, phase):
    sh = wl.shape
    if phase == E.PHASE_EXPERTS:
        return (oracle.expert_arena_bytes(sh, wl.old.placement),
                oracle.expert_arena_bytes(sh, wl.new.placement))
    if phase == E.PHASE_ATTN:
        return oracle.attn_arena_bytes(sh, wl.old.tp), oracle.attn_arena_bytes(sh, wl.new.tp)
    return (oracle.kv_arena_bytes(sh, wl.old.tp, wl.old.kv_num_blocks),
            oracle.kv_arena_bytes(sh, wl.new.tp, wl.new.kv_num_blocks))


@pytest.mark.parametrize("name", ["c1_tiny", "c2_mid", "c3_fine", "c4_large"])
@pytest.mark.parametrize("inverse", [False, True])
def test_segment_replay_equals_oracle(name, inverse):
    wl = small(name)
    if inverse:
        wl = wl.swapped()
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        for phase in range(3):
            so, sn = oracle_sizes(wl, phase)
            assert plan.arena_bytes(phase, E.SIDE_OLD) == so
            assert plan.arena_bytes(phase, E.SIDE_NEW) == sn
            src = arenas(so, 20 + phase)
            want = [np.full(n, FILL, np.uint8) for n in sn]
            got = [np.full(n, FILL, np.uint8) for n in sn]
            run_oracle(wl, phase, src, want)
            segs = plan.segments(phase)
            replay(segs, src, got)
            for r in range(len(sn)):
                assert np.array_equal(got[r], want[r]), (name, phase, r)
            # conservation and exact tiling of the written set
            st = plan.stats(phase)
            assert st["bytes_moved"] == int((segs["run_bytes"] * segs["n_runs"]).sum())
            cover = [np.zeros(n, np.uint8) for n in sn]
            for s in segs:
                for i in range(int(s["n_runs"])):
                    b = int(s["dst_off"]) + i * int(s["dst_pitch"])
                    assert b + int(s["run_bytes"]) <= sn[int(s["dst_rank"])]
                    cover[int(s["dst_rank"])][b:b + int(s["run_bytes"])] += 1
            assert all(c.max(initial=0) <= 1 for c in cover)      # destinations disjoint
            assert sum(int(c.sum()) for c in cover) == st["bytes_moved"]
            if phase != E.PHASE_KV:
                assert all(c.min(initial=1) == 1 for c in cover)  # weights: fully written


def test_replicated_source_is_read_once():
    wl = small("c3_fine")
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        st = plan.stats(E.PHASE_EXPERTS)
        segs = plan.segments(E.PHASE_EXPERTS)
    # every old copy is read exactly once although 12 ranks receive the shared experts
    assert st["bytes_read"] == sum(oracle.expert_arena_bytes(wl.shape, wl.old.placement))
    assert st["bytes_moved"] == sum(oracle.expert_arena_bytes(wl.shape, wl.new.placement))
    groups = np.bincount(segs["group"])
    assert groups.max() == 5       # old rank 0's shared copy feeds new ranks 0, 8, 9, 10, 11


def test_contiguous_placement_coalesces_slots():
    wl = small("c2_mid")
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        segs = plan.segments(E.PHASE_EXPERTS)
    m = wl.shape.d_model * wl.shape.d_ff * wl.shape.elem_bytes
    # EP4 (15 per rank) -> EP6 (10 per rank): 8 strided segments of 5 or 10 experts
    assert len(segs) == 8
    assert sorted(set(int(x) // m for x in segs["run_bytes"])) == [5, 10]


def test_identity_plan_is_one_run_per_arena():
    wl = small("c2_mid")
    with E.Plan(wl.shape, wl.old, wl.old, host_only=True) as plan:
        for phase in (E.PHASE_EXPERTS, E.PHASE_ATTN):
            segs = plan.segments(phase)
            assert (segs["n_runs"] == 1).all()
            assert list(segs["run_bytes"]) == plan.arena_bytes(phase, E.SIDE_OLD)


def test_phases_that_stay_in_place_are_flagged_for_zero_copy():
    """Sec. 5.2: with TP kept, attention weights and KV cache are used where they are.  The plan
    flags a phase as identity exactly when old and new agree on everything that phase sees."""
    wl = small("c2_mid")
    with E.Plan(wl.shape, wl.old, wl.old, host_only=True) as plan:
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [True, True, True]
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:       # EP and the KV tables change, TP kept
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [False, True, False]
    w4 = small("c4_large")                                               # TP 2 -> 4 as well
    with E.Plan(w4.shape, w4.old, w4.new, host_only=True) as plan:
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [False, False, False]
    # the paper's own step: experts re-placed, TP and the KV table kept
    import dataclasses
    kept = dataclasses.replace(wl.new, kv_num_blocks=wl.old.kv_num_blocks, block_table=wl.old.block_table)
    with E.Plan(wl.shape, wl.old, kept, host_only=True) as plan:
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [False, True, True]
    # same TP and table but a larger pool: the arenas differ in size, so the KV cache has to be copied
    grown = dataclasses.replace(kept, kv_num_blocks=wl.old.kv_num_blocks + 1)
    with E.Plan(wl.shape, wl.old, grown, host_only=True) as plan:
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [False, True, False]
    # attention onto extra replicas is a copy even with TP kept
    with E.Plan(wl.shape, wl.old, kept, host_only=True, attn_replicas=2) as plan:
        assert not plan.phase_is_identity(E.PHASE_ATTN)


# ---- validation ------------------------------------------------------------------------

def _plan_code(shape, old, new):
    try:
        E.Plan(shape, old, new, host_only=True).close()
        return 0
    except E.EmoeError as e:
        return e.code


def test_validation_codes():
    wl = small("c1_tiny")
    sh, old, new = wl.shape, wl.old, wl.new
    R = dataclasses.replace
    assert _plan_code(sh, old, new) == 0
    assert _plan_code(R(sh, d_model=0), old, new) == 2                      # SHAPE
    assert _plan_code(sh, old, R(new, tp=3)) == 2                           # 3 does not divide 8
    assert _plan_code(sh, old, R(new, tp=16)) == 2                          # 16 does not divide the 8 q heads
    wide = R(sh, n_q_heads=48)
    assert _plan_code(wide, old, R(new, tp=16)) == 0                        # 8 KV heads on 16 ranks: 2 ranks per head
    assert _plan_code(wide, old, R(new, tp=12)) == 2                        # 12 is no multiple of 8 KV heads
    assert _plan_code(sh, old, R(new, ep=65, placement=[[0]] * 65)) == 9    # too many ranks
    dup = [list(p) for p in new.placement]; dup[0] = [0, 0]
    assert _plan_code(sh, old, R(new, placement=dup)) == 3                  # duplicate in a rank
    miss = [list(p) for p in new.placement]; miss[0] = miss[0][:1]
    assert _plan_code(sh, old, R(new, placement=miss)) == 3                 # expert lost
    assert _plan_code(sh, R(old, placement=[[0, 1, 2, 3], [4, 5, 6]]), new) == 3  # absent from old
    oob = [list(p) for p in new.placement]; oob[0] = [0, 99]
    assert _plan_code(sh, old, R(new, placement=oob)) == 3
    bt = new.block_table.copy(); bt[0, 0] = bt[1, 0]
    assert _plan_code(sh, old, R(new, block_table=bt)) == 4                 # block used twice
    bt = new.block_table.copy(); bt[0, 0] = new.kv_num_blocks
    assert _plan_code(sh, old, R(new, block_table=bt)) == 4                 # id out of range
    bt = new.block_table.copy(); bt[0, 3] = -1
    assert _plan_code(sh, old, R(new, block_table=bt)) == 4                 # hole in a sequence
    assert _plan_code(sh, old, R(new, seq_lens=[256, 256, 256, 255])) == 4  # sequences differ
    assert _plan_code(sh, old, R(new, block_table=new.block_table[:, :8])) == 4  # table too short


def test_host_only_plan_refuses_to_run():
    wl = small("c1_tiny")
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plan:
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_experts([16] * 2, [16] * 4)
        assert ei.value.code == 8


def test_null_arguments():
    L = E.lib()
    assert L.emoe_plan_create(None, None, None, 1, None) == 1
    L.emoe_plan_destroy(None)   # NULL-safe
    assert E.strerror(6).startswith("source and destination")


def test_library_exports_every_declared_symbol():
    """Every function declared in include/emoe.h is exported by libemoe.so."""
    text = open(os.path.join(ROOT, "include", "emoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(emoe_[a-z_]+)\s*\(", text))
    assert declared == set(E.EXPORTS)
    lib = ctypes.CDLL(E.library_path())
    for name in declared:
        assert hasattr(lib, name), name


def test_more_ranks_than_the_library_supports():
    n = E.MAX_RANKS + 1
    sh = W.Shape(1, n, 0, 8, 8, n, n, 8, 4, 2)
    empty = np.zeros((0, 0), np.int32)
    ok = W.ParallelConfig(1, 1, [list(range(n))], 1, [], empty)
    too_many_ep = W.ParallelConfig(n, 1, W.place_round_robin(n, n), 1, [], empty)
    too_many_tp = W.ParallelConfig(1, n, [list(range(n))], 1, [], empty)
    for bad in (too_many_ep, too_many_tp):
        with pytest.raises(E.EmoeError) as ei:
            E.Plan(sh, ok, bad, host_only=True)
        assert ei.value.code == 9


def test_layout_variants_change_segments_not_sizes():
    wl = small("c4_large")
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plain, \
            E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_w13=True, kv_head_major=True) as var:
        for phase in range(3):
            assert plain.arena_bytes(phase, E.SIDE_NEW) == var.arena_bytes(phase, E.SIDE_NEW)
            assert plain.stats(phase)["bytes_moved"] == var.stats(phase)["bytes_moved"]
        # fused gate|up: two runs per layer instead of three per (layer, projection)
        a, b = plain.segments(E.PHASE_EXPERTS), var.segments(E.PHASE_EXPERTS)
        assert int(a["n_runs"].max()) == 3 * wl.shape.n_layers and int(b["n_runs"].max()) == wl.shape.n_layers
        # head-major KV: every piece is a whole head's tokens (B * hd * b bytes per head)
        kv = var.segments(E.PHASE_KV)
        assert set(int(x) for x in kv["run_bytes"]) == {wl.shape.kv_block_tokens * wl.shape.head_dim
                                                       * wl.shape.elem_bytes}
        # the allocation-free KV entry point has no head-major re-split
        with pytest.raises(E.EmoeError) as ei:
            var.reshard_kv_static([16] * 2, [16] * 4)
        assert ei.value.code == 9


def test_header_is_plain_c_and_usable_from_a_c_program(tmp_path):
    """Compiles tests/c_abi_smoke.c as C99 against include/emoe.h, links it with libemoe.so
    and runs it (host-only plan: no GPU needed)."""
    import shutil
    import subprocess
    if not shutil.which("gcc"):
        pytest.skip("no gcc")
    lib = E.library_path()
    E.lib()
    exe = str(tmp_path / "c_abi_smoke")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c_abi_smoke.c"), "-o", exe, lib,
                           "-Wl,-rpath," + os.path.dirname(lib)])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stdout, out.stderr)
    assert "c abi ok" in out.stdout


def test_host_only_plan_and_its_tuning_make_no_cuda_call():
    """A host-only plan - creation, tuning, local rank, queries - must work in a process
    that cannot see any CUDA device at all."""
    import subprocess
    import sys
    code = r"""
import paper_2510_02613_b200 as E, workloads as W
wl = W.make_workload("c4_large", n_layers=1)
with E.Plan(wl.shape, wl.old, wl.new, host_only=True) as p:
    p.set_tuning(max_ctas=24, bulk_tile_bytes=16384, bulk_stages=8, bw_limit_gbs=1000)
    p.set_tuning(bulk_min_run=1024)
    p.set_local_rank(1)
    assert p.num_launches(E.PHASE_STEP) >= 1
    try:
        p.set_tuning(bulk_tile_bytes=65536, bulk_stages=16)   # does not fit shared memory
    except E.EmoeError as e:
        assert e.code == 1
    else:
        raise SystemExit("oversized ring accepted")
print("ok")
"""
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stderr[-2000:]


@pytest.mark.parametrize("name,c,d", [("c1_tiny", 1, 2), ("c1_tiny", 4, 2), ("c4_large", 2, 4),
                                      ("c4_large", 4, 1), ("c4_large", 2, 8), ("c4_large", 16, 4),
                                      ("c2_mid", 2, 2)])
def test_fused_qkv_segment_replay_equals_oracle(name, c, d):
    """The attention phase with a fused qkv matrix per rank: replayed segments == oracle,
    destinations tile the arena exactly once."""
    wl = small(name)
    wl = dataclasses.replace(wl, fused_qkv=True, old=dataclasses.replace(wl.old, tp=c),
                             new=dataclasses.replace(wl.new, tp=d))
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_qkv=True) as plan, \
            E.Plan(wl.shape, wl.old, wl.new, host_only=True) as plain:
        so, sn = oracle_sizes(wl, E.PHASE_ATTN)
        assert plan.arena_bytes(E.PHASE_ATTN, E.SIDE_NEW) == sn
        src = arenas(so, 31)
        want = [np.full(n, FILL, np.uint8) for n in sn]
        got = [np.full(n, FILL, np.uint8) for n in sn]
        run_oracle(wl, E.PHASE_ATTN, src, want)
        segs = plan.segments(E.PHASE_ATTN)
        replay(segs, src, got)
        for r in range(len(sn)):
            assert np.array_equal(got[r], want[r]), r
        cover = [np.zeros(n, np.uint8) for n in sn]
        for s in segs:
            for i in range(int(s["n_runs"])):
                b = int(s["dst_off"]) + i * int(s["dst_pitch"])
                cover[int(s["dst_rank"])][b:b + int(s["run_bytes"])] += 1
        assert all(cv.min(initial=1) == 1 and cv.max(initial=1) == 1 for cv in cover)
        assert plan.stats(E.PHASE_ATTN)["bytes_moved"] == plain.stats(E.PHASE_ATTN)["bytes_moved"]


def test_fused_qkv_needs_whole_query_groups():
    wl = small("c1_tiny")
    sh = dataclasses.replace(wl.shape, n_q_heads=12, n_kv_heads=8)   # 12 % 8 != 0
    cfg = lambda c: dataclasses.replace(c, tp=1)
    with pytest.raises(E.EmoeError) as ei:
        E.Plan(sh, cfg(wl.old), cfg(wl.new), host_only=True, fused_qkv=True)
    assert ei.value.code == 2


@pytest.mark.parametrize("name", ["c2_mid", "c3_fine", "c4_large"])
@pytest.mark.parametrize("ms", [4, 48])
def test_expert_scales_travel_with_their_matrices_in_one_plan(name, ms):
    """emoe_plan_create_ex with expert_scale_bytes: replayed segments == oracle over the
    whole arena (weights, the gap nobody writes, scales)."""
    wl = small(name)
    wl = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, elem_bytes=1, expert_scale_bytes=ms))
    for w in (wl, wl.swapped()):
        with E.Plan(w.shape, w.old, w.new, host_only=True) as plan:
            so, sn = oracle_sizes(w, E.PHASE_EXPERTS)
            assert plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_OLD) == so
            assert plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_NEW) == sn
            src = arenas(so, 51)
            want = [np.full(n, FILL, np.uint8) for n in sn]
            got = [np.full(n, FILL, np.uint8) for n in sn]
            run_oracle(w, E.PHASE_EXPERTS, src, want)
            replay(plan.segments(E.PHASE_EXPERTS), src, got)
            for r in range(len(sn)):
                assert np.array_equal(got[r], want[r]), r
            m = w.shape.d_model * w.shape.d_ff
            slots = sum(len(p) for p in w.new.placement)
            assert plan.stats(E.PHASE_EXPERTS)["bytes_moved"] == w.shape.n_layers * 3 * slots * (m + ms)


def test_plan_options_are_validated():
    wl = small("c2_mid")
    sh = dataclasses.replace(wl.shape, expert_scale_bytes=8)
    with pytest.raises(E.EmoeError) as ei:
        E.Plan(sh, wl.old, wl.new, host_only=True, fused_w13=True)     # scales + fused gate|up
    assert ei.value.code == 9


@pytest.mark.parametrize("name,c,d,replicas,fused", [("c2_mid", 2, 2, 3, False), ("c4_large", 2, 4, 2, False),
                                                    ("c4_large", 4, 2, 2, True), ("c1_tiny", 1, 1, 9, False)])
def test_attention_onto_several_new_replicas_reads_every_source_once(name, c, d, replicas, fused):
    """emoe_plan_create_ex with attn_new_replicas: replayed segments == oracle on all
    d * replicas arenas; bytes written grow with the replicas, bytes read do not."""
    wl = small(name)
    wl = dataclasses.replace(wl, fused_qkv=fused, attn_replicas=replicas, old=dataclasses.replace(wl.old, tp=c),
                             new=dataclasses.replace(wl.new, tp=d))
    with E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_qkv=fused, attn_replicas=replicas) as plan, \
            E.Plan(wl.shape, wl.old, wl.new, host_only=True, fused_qkv=fused) as one:
        so = oracle.attn_arena_bytes(wl.shape, c)
        sn = oracle.attn_arena_bytes(wl.shape, d) * replicas
        assert plan.num_ranks(E.PHASE_ATTN, E.SIDE_NEW) == d * replicas
        assert plan.num_ranks(E.PHASE_KV, E.SIDE_NEW) == d          # experts and KV are not affected
        assert plan.arena_bytes(E.PHASE_ATTN, E.SIDE_NEW) == sn
        src = arenas(so, 71)
        want = [np.full(n, FILL, np.uint8) for n in sn]
        got = [np.full(n, FILL, np.uint8) for n in sn]
        run_oracle(wl, E.PHASE_ATTN, src, want)
        segs = plan.segments(E.PHASE_ATTN)
        replay(segs, src, got)
        for r in range(len(sn)):
            assert np.array_equal(got[r], want[r]), r
        a, b = plan.stats(E.PHASE_ATTN), one.stats(E.PHASE_ATTN)
        assert a["bytes_moved"] == replicas * b["bytes_moved"] and a["bytes_read"] == b["bytes_read"]
        assert len(set(int(g) for g in segs["group"])) == b["n_segments"]      # one read per source run
    if d > 1:       # d * 64 attention arenas are more than the library takes
        with pytest.raises(E.EmoeError) as ei:
            E.Plan(wl.shape, wl.old, wl.new, host_only=True, attn_replicas=E.MAX_RANKS)
        assert ei.value.code == 9
