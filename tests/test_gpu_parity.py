"""GPU parity: the library's output, through the C ABI, must equal the CPU oracle
byte for byte over whole destination arenas (bit-exact: this is byte movement)."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from workloads import device as WD
from gpu_util import KINDS, check_phase_full, check_phase_layers, check_step_full, make_plan, run_phase

pytestmark = pytest.mark.gpu
R = dataclasses.replace


def test_library_is_loaded_from_the_tree():
    assert E.library_path().endswith("paper_2510_02613_b200/libemoe.so")
    E.lib()


@pytest.mark.parametrize("inverse", [False, True])
def test_c1_tiny_all_phases(inverse):
    wl = W.make_workload("c1_tiny")
    if inverse:
        wl = wl.swapped()
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        for phase in range(3):
            check_phase_full(wl, plan, phase)
        check_step_full(wl, plan)
        assert plan.num_launches(E.PHASE_STEP) == 1     # vector work and KV re-split share a kernel
        plan.set_tuning(serial=2)
        assert plan.num_launches(E.PHASE_STEP) == 2     # ... unless told to keep them apart
        check_step_full(wl, plan)


@pytest.mark.parametrize("name", ["c2_mid", "c3_fine", "c4_large"])
def test_one_layer_cut_all_phases(name):
    """One full-width layer: spans thousands of tiles, every kernel, ragged unit tails."""
    wl = W.make_workload(name, n_layers=1)
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        for phase in range(3):
            check_phase_full(wl, plan, phase)
        check_step_full(wl, plan)
        plan.set_tuning(path=2, max_ctas=20)
        check_step_full(wl, plan)


TUNINGS = [dict(path=1), dict(path=2), dict(bulk_tile_bytes=8192, bulk_stages=3),
           dict(bulk_tile_bytes=65536, bulk_stages=2), dict(max_ctas=3),
           dict(bulk_tile_bytes=16384, bulk_stages=12, max_ctas=296),
           dict(kv_mode=1), dict(kv_mode=2), dict(kv_mode=2, max_ctas=3), dict(kv_order=2),
           dict(kv_order=3, kv_mode=2), dict(kv_order=1, unit_order=1),
           dict(kv_order=3, bulk_tile_bytes=16384), dict(kv_mode=3), dict(kv_mode=3, max_ctas=5),
           dict(kv_mode=3, kv_order=3), dict(kv_mode=4), dict(unit_order=2, path=2),
           dict(unit_order=3, path=2, max_ctas=5), dict(path=2, max_ctas=1),
           dict(serial=1, path=2), dict(serial=2), dict(bw_limit_gbs=300, path=2),
           dict(bw_limit_gbs=4000, path=2, max_ctas=16), dict(bulk_min_run=256, path=2),
           dict(bulk_min_run=1024), dict(wait_limit_us=2000000, path=2), dict(path=3), dict(path=3, max_ctas=8)]


@pytest.mark.parametrize("tuning", TUNINGS, ids=lambda t: "-".join("%s%s" % kv for kv in t.items()))
def test_tunings_do_not_change_the_result(tuning):
    for name in ("c1_tiny", "c4_large"):
        wl = W.make_workload(name, n_layers=2 if name == "c1_tiny" else 1)
        if name == "c4_large":   # keep it quick: fewer blocks, thinner experts
            wl = R(wl, shape=R(wl.shape, d_ff=96))
        with E.Plan(wl.shape, wl.old, wl.new) as plan:
            plan.set_tuning(**tuning)
            for phase in range(3):
                check_phase_full(wl, plan, phase)
            check_step_full(wl, plan)


ODD = [
    # d_model, d_ff, hq, hkv, hd, B, elem_bytes, tp_old, tp_new
    (40, 24, 8, 4, 8, 4, 2, 1, 2),      # 16-byte-aligned but short runs
    (33, 7, 6, 6, 3, 5, 1, 2, 3),       # nothing aligned: byte path
    (12, 10, 4, 4, 6, 3, 2, 4, 2),      # 2/4/8-byte alignments
    (64, 520, 8, 2, 64, 16, 2, 2, 1),   # runs straddle the bulk threshold, ragged tile tails
    (16, 1030, 4, 4, 16, 8, 4, 1, 4),   # fp32 elements
]


@pytest.mark.parametrize("dims", ODD, ids=lambda d: "x".join(map(str, d)))
def test_odd_shapes_and_alignments(dims):
    dm, dff, hq, hkv, hd, B, eb, c, d = dims
    sh = W.Shape(3, 7, 1, dm, dff, hq, hkv, hd, B, eb)
    seq_lens = [3 * B + 1, 1, 2 * B]
    nblk = sum(-(-n // B) for n in seq_lens)
    bo = W.make_block_table(11, seq_lens, B, nblk + 2)
    bn = W.make_block_table(12, seq_lens, B, nblk + 5)
    old = W.ParallelConfig(3, c, W.with_shared(W.place_contiguous(7, 3), [7]), nblk + 2, seq_lens, bo)
    new = W.ParallelConfig(2, d, W.with_shared(W.place_round_robin(7, 2), [7]), nblk + 5, seq_lens, bn)
    wl = W.Workload("odd", sh, old, new, 77)
    for w in (wl, wl.swapped()):
        with E.Plan(w.shape, w.old, w.new) as plan:
            for phase in range(3):
                check_phase_full(w, plan, phase)
            for kv_mode in (1, 2, 3, 4):   # every KV kernel (each falls back where it cannot run)
                plan.set_tuning(kv_mode=kv_mode, kv_order=3)
                check_phase_full(w, plan, E.PHASE_KV)
            check_step_full(w, plan)


def test_replicas_with_different_contents_pick_the_documented_source():
    """Arenas are filled by physical position, so replicas differ: parity then also
    pins the source choice (own rank first, else the smallest rank and slot)."""
    sh = W.Shape(2, 6, 0, 64, 128, 4, 4, 16, 4, 2)
    old = W.ParallelConfig(3, 1, [[0, 1, 2, 5], [2, 3, 0], [4, 5, 1]], 1, [], np.zeros((0, 0), np.int32))
    new = W.ParallelConfig(4, 1, [[5, 0], [0, 2, 3], [1, 4, 2], [0, 1, 2, 3, 4, 5]], 1, [],
                           np.zeros((0, 0), np.int32))
    wl = W.Workload("replicas", sh, old, new, 5)
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        check_phase_full(wl, plan, E.PHASE_EXPERTS)
        check_phase_full(wl, plan, E.PHASE_KV)      # no sequences: nothing is written


def test_round_trip_on_the_gpu_is_identity():
    wl = W.make_workload("c4_large", n_layers=1)
    wl = R(wl, shape=R(wl.shape, d_ff=64))
    with E.Plan(wl.shape, wl.old, wl.new) as fwd, E.Plan(wl.shape, wl.new, wl.old) as bwd:
        for phase in range(3):
            a = WD.alloc_filled(fwd.arena_bytes(phase, E.SIDE_OLD), wl.seed, KINDS[phase])
            b = WD.alloc_const(fwd.arena_bytes(phase, E.SIDE_NEW))
            c = WD.alloc_const(fwd.arena_bytes(phase, E.SIDE_OLD))
            if phase == E.PHASE_KV:   # unmapped blocks are not carried: start c from a
                c = [t.clone() for t in a]
            run_phase(fwd, phase, a, b)
            run_phase(bwd, phase, b, c)
            torch.cuda.synchronize()
            if phase == E.PHASE_EXPERTS:
                # replicas differ by position; compare one copy per expert through the oracle
                continue
            assert all(torch.equal(x, y) for x, y in zip(a, c))


def test_argument_errors_launch_nothing():
    wl = W.make_workload("c1_tiny")
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        so = plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_OLD)
        sn = plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_NEW)
        big = torch.full((sum(so) + sum(sn) + 64,), 0xCD, dtype=torch.uint8, device="cuda")
        src = [big[:so[0]], big[so[0]:so[0] + so[1]]]
        good = [torch.empty(n, dtype=torch.uint8, device="cuda") for n in sn]
        # destination 0 aliases the tail of source 1
        bad = [big[so[0] + so[1] - 16: so[0] + so[1] - 16 + sn[0]]] + good[1:]
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_experts(src, bad)
        assert ei.value.code == 6
        mis = [big[sum(so) + 8: sum(so) + 8 + sn[0]]] + good[1:]
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_experts(src, mis)
        assert ei.value.code == 5
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_experts([0, 0], good)
        assert ei.value.code == 1
        torch.cuda.synchronize()
        assert bool((big == 0xCD).all())


def test_zero_copy_phases_accept_their_own_arenas_and_launch_nothing():
    """Sec. 5.2: with TP and the block table kept, attention weights and KV cache are used in
    place.  Such a phase accepts dst == src and leaves the arenas alone, alone or inside the
    whole step; a partly aliased call is still refused."""
    import dataclasses
    from gpu_util import oracle_phase
    base = W.make_workload("c4_large").with_layers(2)
    kept = dataclasses.replace(base.new, tp=base.old.tp, kv_num_blocks=base.old.kv_num_blocks,
                               block_table=base.old.block_table)
    wl = dataclasses.replace(base, new=kept)
    with make_plan(wl) as plan:
        assert [plan.phase_is_identity(ph) for ph in range(3)] == [False, True, True]
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        before = [[t.clone() for t in g] for g in src]
        plan.reshard_attn(src[1], src[1])
        plan.reshard_kv(src[2], src[2])
        dst0 = WD.alloc_const(plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_NEW))
        plan.reshard_step(src, [dst0, src[1], src[2]])
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        for ph in (1, 2):
            h = [t.cpu().numpy() for t in before[ph]]
            want = [a.copy() for a in h]
            oracle_phase(wl, ph, h, want)          # the oracle on a copy of the input changes nothing either
            for g, w, x in zip(src[ph], want, h):
                assert np.array_equal(w, x) and np.array_equal(g.cpu().numpy(), x)
        want = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst0]
        oracle_phase(wl, 0, [t.cpu().numpy() for t in src[0]], want)
        for g, w in zip(dst0, want):
            assert np.array_equal(g.cpu().numpy(), w)
        # one rank aliased, the other not: not the zero-copy case
        other = torch.empty_like(src[2][1])
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_kv(src[2], [src[2][0], other])
        assert ei.value.code == 6
        # a phase that does move bytes never accepts its own arenas
        with pytest.raises(E.EmoeError) as ei:
            plan.reshard_experts(src[0], src[0][:1] + dst0[1:])
        assert ei.value.code == 6
        # one rank per process: only the local rank's arena is looked at
        plan.set_local_rank(1)
        plan.reshard_kv([None, src[2][1]], [None, src[2][1]])
        plan.reshard_attn([None, src[1][1]], [None, src[1][1]])
        plan.set_local_rank(-1)
        torch.cuda.synchronize()
        for ph in (1, 2):
            assert all(torch.equal(a, b) for a, b in zip(src[ph], before[ph]))
        # and the same phases still copy when given separate arenas
        for ph in (1, 2):
            check_phase_full(wl, plan, ph)


def _step_on_host_buffers(wl, host_step):
    from gpu_util import oracle_phase
    with E.Plan(wl.shape, wl.old, wl.new, host_step=host_step, fused_w13=wl.fused_w13,
                kv_head_major=wl.kv_head_major, fused_qkv=wl.fused_qkv, attn_replicas=wl.attn_replicas) as plan:
        h_src, h_dst, d_src, d_dst, want = [], [], [], [], []
        for phase in range(3):
            so, sn = plan.arena_bytes(phase, E.SIDE_OLD), plan.arena_bytes(phase, E.SIDE_NEW)
            hs = [torch.from_numpy(WD.host_slice(wl.seed, KINDS[phase], r, 0, n)).pin_memory()
                  for r, n in enumerate(so)]
            h_src.append(hs)
            h_dst.append([torch.zeros(n, dtype=torch.uint8).pin_memory() for n in sn])
            d_src.append([torch.empty(n, dtype=torch.uint8, device="cuda") for n in so])
            d_dst.append(WD.alloc_const(sn))
            w = [np.full(n, WD.FILL_BYTE, np.uint8) for n in sn]
            oracle_phase(wl, phase, [t.numpy() for t in hs], w)
            want.append(w)
        torch.cuda.synchronize()      # staging arenas were filled on the default stream
        s = torch.cuda.Stream()
        for _ in range(2):      # twice: the pipelined form reuses the plan's events
            for g in h_dst:
                for t in g:
                    t.zero_()
            plan.reshard_step_host(h_src, h_dst, d_src, d_dst, s)
            s.synchronize()
            for phase in range(3):
                for g, w in zip(h_dst[phase], want[phase]):
                    assert np.array_equal(g.numpy(), w)
        assert plan.device_status() == 0


@pytest.mark.parametrize("host_step", [False, True], ids=["serial", "pipelined"])
def test_step_on_host_buffers_matches_oracle(host_step):
    _step_on_host_buffers(W.make_workload("c1_tiny"), host_step)


def test_host_step_with_layout_options():
    """The host-buffer step with attention replicas and a fused qkv matrix (pipelined), and
    with scale tensors (whose arenas are not layer-major: the step then runs serially)."""
    wl = W.make_workload("c1_tiny", n_layers=6)
    _step_on_host_buffers(R(wl, attn_replicas=3, fused_qkv=True), True)
    scaled = R(wl, shape=R(wl.shape, elem_bytes=1, expert_scale_bytes=40))
    _step_on_host_buffers(scaled, True)
    _step_on_host_buffers(scaled, False)


def test_pipelined_host_step_with_a_ragged_last_chunk():
    """35 layers: chunks of 2 layers and a tail chunk of 1."""
    wl = W.make_workload("c1_tiny", n_layers=35)
    wl = R(wl, shape=R(wl.shape, d_ff=64))
    _step_on_host_buffers(wl, True)
    _step_on_host_buffers(wl.swapped(), True)


@pytest.mark.parametrize("name", ["c2_mid", "c3_fine", "c4_large"])
def test_full_size_configs_every_layer(name):
    """The benchmark's launch configuration at full size - the whole step through
    emoe_reshard_step with all arenas resident; EVERY layer compared in full with the
    oracle (layers are independent in every phase, so the oracle takes them one by one)."""
    wl = W.make_workload(name)
    L = wl.shape.n_layers
    torch.cuda.empty_cache()
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        dst = [WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)]
        plan.reshard_step(src, dst)
        torch.cuda.synchronize()
        assert plan.device_status() == 0
        for phase in range(3):
            check_phase_layers(wl, plan, phase, src[phase], dst[phase], range(L))
        # and the per-phase entry points write the same bytes
        for phase in (E.PHASE_ATTN, E.PHASE_KV):
            again = WD.alloc_const(plan.arena_bytes(phase, E.SIDE_NEW))
            run_phase(plan, phase, src[phase], again)
            torch.cuda.synchronize()
            assert all(torch.equal(a, b) for a, b in zip(again, dst[phase]))
            del again
        del src, dst
    torch.cuda.empty_cache()


def _victim_graph(wl, expert_arena, stream, n_layers):
    """The overlap case's concurrent kernel: a grouped expert GEMM (torch.bmm, a fixture of
    the test and of the benchmark, not part of the library) reading expert weights of old
    rank 0, captured as a CUDA graph on `stream`."""
    v = wl.victim
    A, T, D, F = v["active_experts"], v["tokens"], v["d_model"], v["d_ff"]
    slab = expert_arena.view(torch.bfloat16).view(n_layers, 3, len(wl.old.placement[0]), D * F)
    x = (torch.randn(A, T, D, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)

    def gemm_step(l):
        wg, wu = slab[l, 0, :A].view(A, D, F), slab[l, 1, :A].view(A, D, F)
        wd = slab[l, 2, :A].view(A, F, D)
        return torch.bmm(torch.bmm(x, wg) * torch.bmm(x, wu), wd)

    with torch.cuda.stream(stream):
        for l in range(n_layers):
            gemm_step(l)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(4):
                gemm_step(i % n_layers)
    torch.cuda.synchronize()
    return graph


@pytest.mark.parametrize("name", ["c5_overlap", "c4_large"])
def test_overlap_config_is_bit_exact_beside_a_live_gemm(name):
    """The overlap configuration: the reshard on a least-priority stream while a grouped
    expert GEMM keeps running on a high-priority stream, for the default CTA budget and
    for 96 / 48 / 24 CTAs and a bandwidth limit.  Whole destination arenas against the
    oracle every time; the GEMM must really have overlapped the reshard."""
    n_layers = 2
    wl = W.make_workload(name, n_layers=n_layers)
    if wl.victim is None:
        wl = R(wl, victim=W.make_workload("c5_overlap").victim)
        wl = R(wl, victim=dict(wl.victim, d_ff=wl.shape.d_ff))
    least, greatest = torch.cuda.Stream.priority_range()
    s_low, s_high = torch.cuda.Stream(priority=least), torch.cuda.Stream(priority=greatest)
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        dst = [WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)]
        want = []
        for ph in range(3):
            w = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst[ph]]
            from gpu_util import oracle_phase
            oracle_phase(wl, ph, [t.cpu().numpy() for t in src[ph]], w)
            want.append(w)
        graph = _victim_graph(wl, src[0][0], s_high, n_layers)
        for tuning in (dict(), dict(max_ctas=96), dict(max_ctas=48), dict(max_ctas=24),
                       dict(bw_limit_gbs=3000), dict(max_ctas=48, bw_limit_gbs=1500, bulk_stages=3)):
            plan.set_tuning(**tuning)
            for g in dst:
                for t in g:
                    t.fill_(WD.FILL_BYTE)
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            with torch.cuda.stream(s_high):
                ev[0].record(s_high)
                for _ in range(10):
                    graph.replay()
            ev[2].record(s_low)
            plan.reshard_step(src, dst, s_low)
            ev[3].record(s_low)
            with torch.cuda.stream(s_high):
                for _ in range(60):
                    graph.replay()
                ev[1].record(s_high)
            torch.cuda.synchronize()
            # the reshard started before the GEMM loop ended and ended after it had started
            assert ev[0].elapsed_time(ev[3]) > 0 and ev[2].elapsed_time(ev[1]) > 0, tuning
            assert plan.device_status() == 0
            for ph in range(3):
                for r, (t, w) in enumerate(zip(dst[ph], want[ph])):
                    assert np.array_equal(t.cpu().numpy(), w), (tuning, ph, r)


def test_expired_device_wait_is_reported_and_the_plan_recovers():
    """Every device-side wait is bounded.  wait_limit_us = -1 makes the first wait that is not
    already satisfied expire: the kernel must return by itself, the call and the following
    synchronise must succeed, the status word must read EMOE_ERR_DEVICE_TIMEOUT (the output
    of that launch is undefined and is not looked at), and after the word has been cleared
    the same plan - and a fresh one - must be bit-exact again."""
    wl = W.make_workload("c1_tiny")
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        plan.set_tuning(path=2, wait_limit_us=-1)           # forced onto the ring kernel
        so, sn = plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_OLD), plan.arena_bytes(E.PHASE_EXPERTS, E.SIDE_NEW)
        src = WD.alloc_filled(so, wl.seed, W.KIND_EXPERTS)
        dst = WD.alloc_const(sn)
        plan.reshard_experts(src, dst)
        torch.cuda.synchronize()                            # returns: no trap, no endless spin
        assert plan.device_status() == 10
        plan.clear_device_status()
        assert plan.device_status() == 0
        plan.set_tuning(path=2)                             # default bound again
        for phase in range(3):
            check_phase_full(wl, plan, phase)
        # the staged and the tensor-map KV kernels have the same bounded waits
        for kv_mode in (2, 3):
            plan.set_tuning(kv_mode=kv_mode, wait_limit_us=-1)
            ko, kn = plan.arena_bytes(E.PHASE_KV, E.SIDE_OLD), plan.arena_bytes(E.PHASE_KV, E.SIDE_NEW)
            ks, kd = WD.alloc_filled(ko, wl.seed, W.KIND_KV), WD.alloc_const(kn)
            plan.reshard_kv(ks, kd)
            torch.cuda.synchronize()
            assert plan.device_status() == 10
            plan.clear_device_status()
            plan.set_tuning(kv_mode=kv_mode)
            check_phase_full(wl, plan, E.PHASE_KV)
    with E.Plan(wl.shape, wl.old, wl.new) as fresh:
        check_step_full(wl, fresh)


def test_maximum_rank_counts():
    """EMOE_MAX_RANKS = 64 ranks on both sides of every phase: EP 64 -> 63 with replicas,
    TP 1 -> 64 and back (64 KV heads, one per rank)."""
    n = E.MAX_RANKS
    sh = W.Shape(1, 2 * n, 1, 16, 8, n, n, 8, 4, 2)
    seq_lens = [9, 4]
    nblk = sum(-(-x // 4) for x in seq_lens)
    bo = W.make_block_table(21, seq_lens, 4, nblk)
    bn = W.make_block_table(22, seq_lens, 4, nblk + 3)
    old = W.ParallelConfig(n, 1, W.with_shared(W.place_round_robin(2 * n, n), [2 * n]), nblk, seq_lens, bo)
    new = W.ParallelConfig(n - 1, n, W.with_shared(W.place_contiguous(2 * n, n - 1), [2 * n]),
                           nblk + 3, seq_lens, bn)
    wl = W.Workload("max_ranks", sh, old, new, 9)
    for w in (wl, wl.swapped()):
        with E.Plan(w.shape, w.old, w.new) as plan:
            for kv_mode in (1, 2, 3):
                plan.set_tuning(kv_mode=kv_mode)
                for phase in range(3):
                    check_phase_full(w, plan, phase)
            check_step_full(w, plan)   # 64 + 63 + .. ranks do not fit one launch set: falls back


@pytest.mark.parametrize("c,d", [(2, 8), (8, 4), (4, 16), (16, 8), (8, 8)])
def test_more_tp_ranks_than_kv_heads(c, d):
    """Large-expert-count shape (4 KV heads, 32 q heads) at TP degrees above the KV head
    count: every head is held by several ranks, attention k/v and the KV cache follow."""
    wl = W.make_workload("c4_large", n_layers=1)
    wl = R(wl, shape=R(wl.shape, d_ff=64, d_model=256), old=R(wl.old, tp=c), new=R(wl.new, tp=d))
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        for phase in (E.PHASE_ATTN, E.PHASE_KV):
            check_phase_full(wl, plan, phase)
        for kv_mode in (2, 3, 4):
            plan.set_tuning(kv_mode=kv_mode, max_ctas=7)
            check_phase_full(wl, plan, E.PHASE_KV)
        st = plan.stats(E.PHASE_KV)
        used = sum(-(-n // 16) for n in wl.old.seq_lens)
        assert st["bytes_moved"] == 2 * used * 16 * max(4, d) * 128 * 2


@pytest.mark.parametrize("name", ["c1_tiny", "c3_fine", "c4_large"])
def test_layout_variants_one_layer(name):
    """Fused gate|up expert tensors and head-major KV blocks at full width."""
    from gpu_util import make_plan
    wl = W.make_workload(name, n_layers=2 if name == "c1_tiny" else 1)
    wl = R(wl, fused_w13=True, kv_head_major=True)
    for w in (wl, wl.swapped()):
        with make_plan(w) as plan:
            for phase in (E.PHASE_EXPERTS, E.PHASE_KV):
                check_phase_full(w, plan, phase)
            plan.set_tuning(path=2, max_ctas=9)
            for phase in (E.PHASE_EXPERTS, E.PHASE_KV):
                check_phase_full(w, plan, phase)


@pytest.mark.parametrize("name,c,d", [("c1_tiny", 1, 2), ("c4_large", 2, 4), ("c4_large", 4, 2),
                                      ("c4_large", 2, 8), ("c4_large", 8, 1), ("c3_fine", 2, 4)])
def test_fused_qkv_layout(name, c, d):
    """Attention re-slice with one fused qkv matrix per rank (rows grouped by KV head), at
    full width, alone and as part of the whole step."""
    from gpu_util import make_plan
    wl = W.make_workload(name, n_layers=2)
    wl = R(wl, fused_qkv=True, old=R(wl.old, tp=c), new=R(wl.new, tp=d),
           shape=R(wl.shape, d_ff=64))
    with make_plan(wl) as plan:
        check_phase_full(wl, plan, E.PHASE_ATTN)
        check_step_full(wl, plan)
        plan.set_tuning(path=2, max_ctas=11)
        check_phase_full(wl, plan, E.PHASE_ATTN)


@pytest.mark.parametrize("name,c,d,replicas", [("c3_fine", 2, 2, 3), ("c4_large", 2, 4, 2), ("c4_large", 4, 2, 5)])
def test_attention_for_added_replicas(name, c, d, replicas):
    """The paper's attention step: added data-parallel replicas receive whole copies of the
    attention shards (here together with a TP change); every replica against the oracle, alone
    and inside the whole step, the shards read once and stored to all replicas."""
    from gpu_util import make_plan
    wl = W.make_workload(name, n_layers=2)
    wl = R(wl, attn_replicas=replicas, old=R(wl.old, tp=c), new=R(wl.new, tp=d), shape=R(wl.shape, d_ff=64))
    with make_plan(wl) as plan:
        assert plan.num_ranks(E.PHASE_ATTN, E.SIDE_NEW) == d * replicas
        check_phase_full(wl, plan, E.PHASE_ATTN)
        check_step_full(wl, plan)
        plan.set_tuning(path=2, max_ctas=7)
        check_phase_full(wl, plan, E.PHASE_ATTN)
        st = plan.stats(E.PHASE_ATTN)
        assert st["bytes_moved"] == replicas * st["bytes_read"]


def test_scaling_sequence_with_chosen_placements():
    """A sequence of scale steps in the paper's step pattern (+2 devices per step, then
    back down), each new placement chosen by emoe_place_min_transfer from the previous
    one; after every step the arenas must equal the oracle applied to the previous arenas."""
    sh = W.Shape(2, 24, 0, 64, 96, 8, 8, 16, 4, 2)
    empty = np.zeros((0, 0), np.int32)
    placement = W.place_contiguous(24, 2)
    cur = WD.alloc_filled(oracle.expert_arena_bytes(sh, placement), 123, W.KIND_EXPERTS)
    for ep_new in (4, 6, 8, 6, 4, 2):
        new_p, kept = E.place_min_transfer(24, placement, ep_new)
        old = W.ParallelConfig(len(placement), 1, placement, 1, [], empty)
        new = W.ParallelConfig(ep_new, 1, new_p, 1, [], empty)
        wl = W.Workload("seq", sh, old, new, 123)
        with E.Plan(sh, old, new) as plan:
            _, nxt = check_phase_full(wl, plan, E.PHASE_EXPERTS, src=cur)
        assert kept == min(len(placement), ep_new) * min(24 // len(placement), 24 // ep_new)
        placement, cur = new_p, nxt


def test_step_captured_in_a_cuda_graph_replays_correctly():
    """The reshard calls only enqueue kernels, so a step can be captured once and replayed;
    every replay must write the oracle's bytes (the destination is re-filled in between)."""
    from gpu_util import oracle_phase
    wl = W.make_workload("c1_tiny")
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        dst = [WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)]
        want = []
        for ph in range(3):
            w = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst[ph]]
            oracle_phase(wl, ph, [t.cpu().numpy() for t in src[ph]], w)
            want.append(w)
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            plan.reshard_step(src, dst, stream)           # warm-up outside the capture
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                plan.reshard_step(src, dst, stream)
            for _ in range(3):
                for g in dst:
                    for t in g:
                        t.fill_(WD.FILL_BYTE)
                graph.replay()
                graph.replay()                            # back to back: same work counters
                stream.synchronize()
                for ph in range(3):
                    for t, w in zip(dst[ph], want[ph]):
                        assert np.array_equal(t.cpu().numpy(), w)
        assert plan.device_status() == 0
    # and a bulk-kernel step (forced), whose launches claim work through the plan's counters
    wl = W.make_workload("c2_mid", n_layers=1)
    wl = R(wl, shape=R(wl.shape, d_ff=128))
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        plan.set_tuning(path=2)
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        dst = [WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)]
        torch.cuda.synchronize()      # the arenas were filled on the default stream
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            plan.reshard_step(src, dst, stream)
            stream.synchronize()
            ref = [[t.clone() for t in g] for g in dst]
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                plan.reshard_step(src, dst, stream)
            for g in dst:
                for t in g:
                    t.fill_(WD.FILL_BYTE)
            for _ in range(6):                            # more replays than counter slots
                graph.replay()
            stream.synchronize()
            for ph in range(3):
                assert all(torch.equal(a, b) for a, b in zip(dst[ph], ref[ph]))
        check_step_full(wl, plan)


def test_kv_delta_plan_recopies_blocks_written_during_the_migration():
    """Scale while serving: migrate the whole KV cache, let "serving" append tokens to the
    last block of every sequence and claim one more block, then re-copy only those blocks
    with a delta plan (every dirty block a one-block sequence).  The result must equal the
    oracle run on the final cache in one go."""
    from gpu_util import oracle_phase
    wl = W.make_workload("c4_large", n_layers=2)
    B = wl.shape.kv_block_tokens
    # leave room for one more block per sequence in both pools
    n_seq = len(wl.old.seq_lens)
    nb_old, nb_new = wl.old.kv_num_blocks + n_seq, wl.new.kv_num_blocks + n_seq
    seq0 = [n - (n % B or B) + 3 for n in wl.old.seq_lens]          # last block partly filled
    def tables(seq_lens):
        return (W.make_block_table(31, seq_lens, B, nb_old), W.make_block_table(32, seq_lens, B, nb_new))
    grown = [n + B for n in seq0]                                    # one more block each
    bo1, bn1 = tables(grown)                                         # final tables; the early ones are their prefix
    nblk0 = [-(-n // B) for n in seq0]
    bo0 = np.full_like(bo1, -1); bn0 = np.full_like(bn1, -1)
    for s_, k in enumerate(nblk0):
        bo0[s_, :k] = bo1[s_, :k]; bn0[s_, :k] = bn1[s_, :k]
    early = R(wl, old=R(wl.old, kv_num_blocks=nb_old, seq_lens=seq0, block_table=bo0),
              new=R(wl.new, kv_num_blocks=nb_new, seq_lens=seq0, block_table=bn0))
    final = R(wl, old=R(wl.old, kv_num_blocks=nb_old, seq_lens=grown, block_table=bo1),
              new=R(wl.new, kv_num_blocks=nb_new, seq_lens=grown, block_table=bn1))
    # dirty blocks: the last block of the early state and the new block, per sequence
    d_old = np.array([[bo1[s_, k - 1]] for s_, k in enumerate(nblk0)] + [[bo1[s_, k]] for s_, k in enumerate(nblk0)], np.int32)
    d_new = np.array([[bn1[s_, k - 1]] for s_, k in enumerate(nblk0)] + [[bn1[s_, k]] for s_, k in enumerate(nblk0)], np.int32)
    delta = R(wl, old=R(wl.old, kv_num_blocks=nb_old, seq_lens=[B] * len(d_old), block_table=d_old),
              new=R(wl.new, kv_num_blocks=nb_new, seq_lens=[B] * len(d_new), block_table=d_new))
    with E.Plan(early.shape, early.old, early.new) as p_all, E.Plan(delta.shape, delta.old, delta.new) as p_delta:
        src = WD.alloc_filled(p_all.arena_bytes(E.PHASE_KV, E.SIDE_OLD), wl.seed, W.KIND_KV)
        dst = WD.alloc_const(p_all.arena_bytes(E.PHASE_KV, E.SIDE_NEW))
        p_all.reshard_kv(src, dst)
        # serving writes: new contents for every dirty block of every layer and K|V
        L, hl = wl.shape.n_layers, wl.shape.n_kv_heads // wl.old.tp
        blk = B * hl * wl.shape.head_dim * wl.shape.elem_bytes
        for t in src:
            pool = t.view(L * 2, nb_old, blk)
            pool[:, torch.from_numpy(d_old[:, 0].astype(np.int64)).cuda()] += 1
        p_delta.reshard_kv(src, dst)
        torch.cuda.synchronize()
        want = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst]
        oracle_phase(final, E.PHASE_KV, [t.cpu().numpy() for t in src], want)
        for r, (g, w) in enumerate(zip(dst, want)):
            assert np.array_equal(g.cpu().numpy(), w), "rank %d" % r
        moved = p_delta.stats(E.PHASE_KV)["bytes_moved"]
        assert moved * 8 < p_all.stats(E.PHASE_KV)["bytes_moved"]      # the delta is small


@pytest.mark.parametrize("name", ["c2_mid", "c4_large"])
def test_one_plan_on_several_streams_at_once(name):
    """The header allows up to four launches of one phase of one plan in flight at once (they
    claim work through per-launch counters) and whole-step calls from several streams (they
    share the plan's side stream).  Three streams run the same step into three sets of
    destination arenas without any ordering between them, twice over; every set must equal
    the oracle."""
    from gpu_util import oracle_phase
    wl = W.make_workload(name, n_layers=1)
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
        want = []
        for ph in range(3):
            w = [np.full(n, WD.FILL_BYTE, np.uint8) for n in plan.arena_bytes(ph, E.SIDE_NEW)]
            oracle_phase(wl, ph, [t.cpu().numpy() for t in src[ph]], w)
            want.append(w)
        sets = [[WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)] for _ in range(3)]
        streams = [torch.cuda.Stream() for _ in range(3)]
        torch.cuda.synchronize()
        for tuning in (dict(), dict(path=2, max_ctas=20)):
            plan.set_tuning(**tuning)
            for dst in sets:
                for g in dst:
                    for t in g:
                        t.fill_(WD.FILL_BYTE)
            torch.cuda.synchronize()
            for rounds in range(2):
                for st, dst in zip(streams, sets):
                    plan.reshard_step(src, dst, st)
                for st, dst in zip(streams, sets):          # and the per-phase calls on top
                    plan.reshard_experts(src[0], dst[0], st)
                torch.cuda.synchronize()                    # at most four unfinished launches per phase
            assert plan.device_status() == 0
            for k, dst in enumerate(sets):
                for ph in range(3):
                    for r, (t, w) in enumerate(zip(dst[ph], want[ph])):
                        assert np.array_equal(t.cpu().numpy(), w), (tuning, k, ph, r)


def test_kv_migration_while_a_second_stream_appends_tokens():
    """Scale while serving, for real this time: the whole-cache migration runs on one stream
    WHILE a second stream keeps appending tokens to the last block of every sequence (the
    writes race with the copy of those blocks, so their destination bytes are undefined for
    the moment); afterwards a delta plan that lists just the blocks written re-copies them.
    The final cache must equal the oracle run on the final source in one go, and the two
    streams must really have overlapped in time."""
    from gpu_util import oracle_phase
    wl = W.make_workload("c4_large", n_layers=8)
    B, L = wl.shape.kv_block_tokens, wl.shape.n_layers
    hl = wl.shape.n_kv_heads // wl.old.tp
    blk = B * hl * wl.shape.head_dim * wl.shape.elem_bytes
    nblk = [-(-n // B) for n in wl.old.seq_lens]
    last_old = np.array([[wl.old.block_table[s_, k - 1]] for s_, k in enumerate(nblk)], np.int32)
    last_new = np.array([[wl.new.block_table[s_, k - 1]] for s_, k in enumerate(nblk)], np.int32)
    delta = R(wl, old=R(wl.old, seq_lens=[B] * len(nblk), block_table=last_old),
              new=R(wl.new, seq_lens=[B] * len(nblk), block_table=last_new))
    idx = torch.from_numpy(last_old[:, 0].astype(np.int64)).cuda()
    s_copy, s_serve = torch.cuda.Stream(), torch.cuda.Stream()
    with E.Plan(wl.shape, wl.old, wl.new) as p_all, E.Plan(delta.shape, delta.old, delta.new) as p_delta:
        src = WD.alloc_filled(p_all.arena_bytes(E.PHASE_KV, E.SIDE_OLD), wl.seed, W.KIND_KV)
        dst = WD.alloc_const(p_all.arena_bytes(E.PHASE_KV, E.SIDE_NEW))
        pools = [t.view(L * 2, wl.old.kv_num_blocks, blk) for t in src]
        torch.cuda.synchronize()
        overlapped = False
        for attempt in range(4):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record(s_copy)
            for _ in range(4):                    # the migration, a few times over to make it last
                p_all.reshard_kv(src, dst, s_copy)
            ev[1].record(s_copy)
            with torch.cuda.stream(s_serve):
                ev[2].record(s_serve)
                for step in range(40):            # "decode steps": one more token per sequence each
                    for pool in pools:
                        pool[:, idx, (step % B) * hl * 8:(step % B) * hl * 8 + 8] += 1
                ev[3].record(s_serve)
            torch.cuda.synchronize()
            # serving started before the migration ended and the migration started before serving ended
            overlapped = ev[2].elapsed_time(ev[1]) > 0 and ev[0].elapsed_time(ev[3]) > 0
            if overlapped:
                break
        assert overlapped, "the appending stream never ran beside the migration"
        p_delta.reshard_kv(src, dst, s_copy)      # close the gap: only the blocks written since
        s_copy.synchronize()
        want = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst]
        oracle_phase(wl, E.PHASE_KV, [t.cpu().numpy() for t in src], want)
        for r, (g, w) in enumerate(zip(dst, want)):
            assert np.array_equal(g.cpu().numpy(), w), "rank %d" % r
        assert p_delta.stats(E.PHASE_KV)["bytes_moved"] * 20 < p_all.stats(E.PHASE_KV)["bytes_moved"]
        assert p_all.device_status() == 0 and p_delta.device_status() == 0


def test_fp8_weights_with_block_scales_in_one_plan():
    """FP8 expert weights (elem_bytes = 1) and their per-128x128-block fp32 scale tensors
    ([d_ff/128][d_model/128] floats per matrix) move with the same placement through ONE plan
    and one call: the arena of a rank holds the weights and, after them, the scales."""
    base = W.make_workload("c3_fine", n_layers=2)
    scale_bytes = (base.shape.d_model // 128) * (base.shape.d_ff // 128) * 4
    assert scale_bytes == 16 * 11 * 4
    wl = R(base, shape=R(base.shape, elem_bytes=1, expert_scale_bytes=scale_bytes))
    for w in (wl, wl.swapped()):
        with E.Plan(w.shape, w.old, w.new) as plan:
            check_phase_full(w, plan, E.PHASE_EXPERTS)
            check_step_full(w, plan)
            assert plan.num_launches(E.PHASE_STEP) <= 2
            plan.set_tuning(path=2, max_ctas=13)
            check_phase_full(w, plan, E.PHASE_EXPERTS)
            plan.set_tuning(path=1)
            check_phase_full(w, plan, E.PHASE_EXPERTS)
    # odd sizes: scale tensors that are not multiples of 16 bytes
    odd = R(base, shape=R(base.shape, n_layers=3, d_model=24, d_ff=20, elem_bytes=1, expert_scale_bytes=6))
    with E.Plan(odd.shape, odd.old, odd.new) as plan:
        check_phase_full(odd, plan, E.PHASE_EXPERTS)
        check_step_full(odd, plan)
