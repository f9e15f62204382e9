"""Plan cache over a scaling sequence, and the compacting KV block table."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest

import oracle
import paper_2510_02613_b200 as E
import workloads as W

R = dataclasses.replace
EMPTY = np.zeros((0, 0), np.int32)


def weights_cfg(placement, tp):
    return W.ParallelConfig(len(placement), tp, placement, 1, [], EMPTY)


def test_plan_cache_over_an_oscillating_scaling_sequence():
    """2 -> 4 -> 6 -> 8 -> 6 -> 4 -> 2 devices and the same climb again: the second pass
    reuses every plan of the first."""
    sh = W.Shape(2, 24, 0, 16, 8, 8, 8, 4, 4, 2)
    seq = [2, 4, 6, 8, 6, 4, 2, 4, 6, 8, 6, 4, 2]
    with E.PlanCache(capacity=8) as cache:
        hits = []
        for a, b in zip(seq, seq[1:]):
            old = weights_cfg(W.place_contiguous(24, a), 2 if a < 6 else 4)
            new = weights_cfg(W.place_contiguous(24, b), 2 if b < 6 else 4)
            plan, hit = cache.get(sh, old, new, host_only=True)
            hits.append(hit)
            assert plan.stats(E.PHASE_EXPERTS)["bytes_moved"] == 2 * 3 * 24 * 16 * 8 * 2
        assert hits == [False] * 6 + [True] * 6
        assert cache.stats() == dict(hits=6, misses=6, evictions=0, size=6)
        # the same inputs give the same plan object; different flags or one id swapped do not
        old, new = weights_cfg(W.place_contiguous(24, 2), 2), weights_cfg(W.place_contiguous(24, 4), 2)
        p1, h1 = cache.get(sh, old, new, host_only=True)
        p2, h2 = cache.get(sh, old, new, host_only=True)
        assert h1 and h2 and p1._h.value == p2._h.value
        _, h3 = cache.get(sh, old, new, host_only=True, fused_w13=True)
        swapped = [list(p) for p in new.placement]
        swapped[0][0], swapped[1][0] = swapped[1][0], swapped[0][0]
        _, h4 = cache.get(sh, old, weights_cfg(swapped, 2), host_only=True)
        assert not h3 and not h4


def test_plan_cache_evicts_the_least_recently_used_plan_and_reports_errors():
    sh = W.Shape(1, 8, 0, 16, 8, 8, 8, 4, 4, 2)
    cfgs = [weights_cfg(W.place_contiguous(8, n), 1) for n in (1, 2, 4, 8)]
    with E.PlanCache(capacity=2) as cache:
        cache.get(sh, cfgs[0], cfgs[1], host_only=True)
        cache.get(sh, cfgs[1], cfgs[2], host_only=True)
        cache.get(sh, cfgs[0], cfgs[1], host_only=True)           # refreshes the first
        cache.get(sh, cfgs[2], cfgs[3], host_only=True)           # evicts 1 -> 2
        assert cache.stats() == dict(hits=1, misses=3, evictions=1, size=2)
        assert cache.get(sh, cfgs[0], cfgs[1], host_only=True)[1]
        assert not cache.get(sh, cfgs[1], cfgs[2], host_only=True)[1]
        bad = weights_cfg([[0, 1, 2, 3], [4, 5, 6]], 1)          # expert 7 missing
        with pytest.raises(E.EmoeError) as ei:
            cache.get(sh, cfgs[0], bad, host_only=True)
        assert ei.value.code == 3
        assert cache.stats()["size"] == 2                        # errors are not stored


def test_plan_cache_keys_on_the_mapped_block_table_entries_only():
    wl = W.make_workload("c1_tiny")
    with E.PlanCache(capacity=4) as cache:
        assert not cache.get(wl.shape, wl.old, wl.new, host_only=True)[1]
        wider = np.full((wl.new.block_table.shape[0], wl.new.block_table.shape[1] + 3), -1, np.int32)
        wider[:, :wl.new.block_table.shape[1]] = wl.new.block_table
        assert cache.get(wl.shape, wl.old, R(wl.new, block_table=wider), host_only=True)[1]   # padding differs
        moved = wl.new.block_table.copy()
        moved[0, 0], moved[0, 1] = moved[0, 1], moved[0, 0]
        assert not cache.get(wl.shape, wl.old, R(wl.new, block_table=moved), host_only=True)[1]


# ---- compaction -------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(6))
def test_compact_table_equals_the_definition(seed):
    rng = np.random.default_rng(seed)
    B = int(rng.integers(1, 9))
    seq_lens = [int(x) for x in rng.integers(0, 40, size=int(rng.integers(1, 7)))]
    need = sum(-(-n // B) for n in seq_lens)
    nb = need + int(rng.integers(0, 12))
    in_use = [int(x) for x in rng.permutation(nb)[:nb - need]][:int(rng.integers(0, nb - need + 1))]
    got = E.kv_compact_table(B, seq_lens, nb, in_use)
    want = oracle.compact_block_table(seq_lens, B, nb, in_use)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("seed", range(6))
def test_compact_table_in_old_address_order_equals_the_definition(seed):
    rng = np.random.default_rng(100 + seed)
    B = int(rng.integers(1, 9))
    seq_lens = [int(x) for x in rng.integers(0, 40, size=int(rng.integers(1, 7)))]
    need = sum(-(-n // B) for n in seq_lens)
    nb_old, nb = need + int(rng.integers(0, 5)), need + int(rng.integers(0, 12))
    old = W.make_block_table(W.rng.stream_key(seed, 3), seq_lens, B, nb_old) if need else np.zeros((len(seq_lens), 0), np.int32)
    in_use = [int(x) for x in rng.permutation(nb)[:nb - need]][:int(rng.integers(0, nb - need + 1))]
    got = E.kv_compact_table(B, seq_lens, nb, in_use, old_table=old)
    want = oracle.compact_block_table(seq_lens, B, nb, in_use, old_table=old)
    assert np.array_equal(got, want)
    pairs = sorted((int(o), int(n)) for o, n in zip(old.reshape(-1), got.reshape(-1)) if o >= 0)
    assert [n for _, n in pairs] == sorted(n for _, n in pairs)        # old and new ids rise together
    # the set of ids handed out does not depend on the order they are served in
    plain = E.kv_compact_table(B, seq_lens, nb, in_use)
    assert sorted(int(x) for x in got.reshape(-1) if x >= 0) == sorted(int(x) for x in plain.reshape(-1) if x >= 0)


def test_compact_table_properties():
    """What "compacted" means, checked without the oracle: the blocks handed out are exactly
    the n smallest free ids, they increase along (sequence, block), a fresh pool gives the
    identity order, and blocks in use are never handed out."""
    B, seq_lens, nb = 4, [9, 4, 1, 13], 20
    in_use = [0, 3, 4, 11]
    t = E.kv_compact_table(B, seq_lens, nb, in_use)
    flat = [int(x) for row in t for x in row if x >= 0]
    free = [x for x in range(nb) if x not in in_use]
    assert flat == free[:len(flat)] and len(flat) == 3 + 1 + 1 + 4
    assert [int((row >= 0).sum()) for row in t] == [3, 1, 1, 4]
    fresh = E.kv_compact_table(B, seq_lens, nb)
    assert [int(x) for row in fresh for x in row if x >= 0] == list(range(9))
    assert np.array_equal(oracle.compact_block_table(seq_lens, B, nb), fresh)
    with pytest.raises(E.EmoeError) as ei:
        E.kv_compact_table(B, seq_lens, 10, [0, 1])               # 8 free blocks, 9 needed
    assert ei.value.code == 11
    with pytest.raises(E.EmoeError) as ei:
        E.kv_compact_table(B, seq_lens, nb, [3, 3])
    assert ei.value.code == 4
    with pytest.raises(ValueError):
        oracle.compact_block_table(seq_lens, B, 10, [0, 1])


# ---- GPU --------------------------------------------------------------------------------

@pytest.mark.gpu
def test_gpu_scale_down_compacts_the_kv_cache_into_a_pool_that_is_partly_in_use():
    """TP4 -> TP2 scale-down of the large-expert-count shape: the destination pool already
    holds blocks of sequences the surviving instance serves (marked in use, pre-filled with
    their own bytes); the migrated blocks must fill the lowest free ids and nothing else may
    change.  Whole arenas against the oracle."""
    import torch
    from gpu_util import check_phase_full
    wl = W.make_workload("c4_large", n_layers=2).swapped()
    B = wl.shape.kv_block_tokens
    need = sum(-(-n // B) for n in wl.old.seq_lens)
    nb_new = need + 300
    in_use = [int(x) for x in W.rng.permutation(W.rng.stream_key(5, 9), nb_new)[:300]]
    table = E.kv_compact_table(B, wl.old.seq_lens, nb_new, in_use)
    assert np.array_equal(table, oracle.compact_block_table(wl.old.seq_lens, B, nb_new, in_use))
    wl = R(wl, new=R(wl.new, kv_num_blocks=nb_new, block_table=table))
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        check_phase_full(wl, plan, E.PHASE_KV)


@pytest.mark.gpu
def test_gpu_cached_plans_over_a_sequence_that_changes_ep_tp_and_moves_kv():
    """2 -> 4 -> 8 -> 4 -> 2 devices twice over, TP following the device count, the KV cache
    moved and compacted at every step; every step through a cached plan against the oracle,
    the second pass entirely from the cache."""
    import torch
    from gpu_util import KINDS, oracle_phase
    from workloads import device as WD
    sh = W.Shape(2, 16, 0, 64, 96, 8, 8, 16, 4, 2)
    seq_lens = [37, 5, 64, 18]
    need = sum(-(-n // 4) for n in seq_lens)
    def cfg(n_dev):
        table = E.kv_compact_table(4, seq_lens, need + n_dev, list(range(0, n_dev)))
        return W.ParallelConfig(n_dev, min(n_dev, 8), W.place_contiguous(16, n_dev), need + n_dev,
                                seq_lens, table)
    seq = [2, 4, 8, 4, 2, 4, 8, 4, 2]
    with E.PlanCache(capacity=8) as cache:
        hits = []
        for a, b in zip(seq, seq[1:]):
            wl = W.Workload("seq", sh, cfg(a), cfg(b), 77)
            plan, hit = cache.get(wl.shape, wl.old, wl.new)
            hits.append(hit)
            src = [WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, KINDS[ph]) for ph in range(3)]
            dst = [WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)) for ph in range(3)]
            plan.reshard_step(src, dst)
            torch.cuda.synchronize()
            assert plan.device_status() == 0
            for ph in range(3):
                want = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst[ph]]
                oracle_phase(wl, ph, [t.cpu().numpy() for t in src[ph]], want)
                for r, (g, w) in enumerate(zip(dst[ph], want)):
                    assert np.array_equal(g.cpu().numpy(), w), (a, b, ph, r)
        assert hits == [False] * 4 + [True] * 4
