"""Paged expert store on the GPU: after every scale step the pool's ranges, read back as
dense arenas, must equal the oracle's expert re-pack of the previous dense arenas byte
for byte; the step's statistics must match the host-side dry run."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from helpers import rand_bytes

pytestmark = pytest.mark.gpu


def dense_sizes(sh, placement):
    return oracle.expert_arena_bytes(sh, placement)


def read_pool(pool, sh, placement):
    out = [np.zeros(n, np.uint8) for n in dense_sizes(sh, placement)]
    for r, a in enumerate(out):
        if a.size:
            pool.read(r, a)
    torch.cuda.synchronize()
    return out


def run_chain(sh, placements, key=50):
    """Creates the pool with placements[0], then steps through the others."""
    cur = [rand_bytes((key, r), n) for r, n in enumerate(dense_sizes(sh, placements[0]))]
    torch.cuda.empty_cache()      # pages come from the driver, not from torch's cache
    with E.VmmPool(sh, placements[0]) as pool:
        for r, a in enumerate(cur):
            if a.size:
                pool.write(r, a)
        torch.cuda.synchronize()
        assert all(np.array_equal(x, y) for x, y in zip(read_pool(pool, sh, placements[0]), cur))
        for old_p, new_p in zip(placements, placements[1:]):
            info = pool.arena(0)
            want_stats = E.vmm_dry_run(sh, old_p, new_p, info["slab_bytes"])
            st = pool.reshard(new_p)
            for k in ("slabs_remapped", "slabs_copied", "bytes_copied", "bytes_read", "physical_bytes"):
                assert st[k] == want_stats[k], k
            want = [np.zeros(n, np.uint8) for n in dense_sizes(sh, new_p)]
            oracle.reshard_experts(sh, old_p, new_p, cur, want)
            assert pool.num_ranks() == len(new_p)
            got = read_pool(pool, sh, new_p)
            for r, (g, w) in enumerate(zip(got, want)):
                assert np.array_equal(g, w), "rank %d after %r -> %r" % (r, old_p, new_p)
            for r, p in enumerate(new_p):
                a = pool.arena(r)
                assert a["n_slots"] == len(p) and a["bytes"] == 3 * sh.n_layers * len(p) * a["slab_bytes"]
                assert a["matrix_bytes"] == sh.d_model * sh.d_ff * sh.elem_bytes
                assert a["base"] % 512 == 0
            cur = want
    return True


def test_scale_up_then_down_then_up_again():
    sh = W.Shape(2, 12, 0, 64, 96, 4, 4, 16, 4, 2)     # m = 12 KiB, far below one page
    run_chain(sh, [W.place_contiguous(12, 4), W.place_contiguous(12, 6), W.place_contiguous(12, 2),
                   W.place_round_robin(12, 4), W.place_contiguous(12, 4)])


def test_replicas_shared_experts_and_scrambled_slots():
    sh = W.Shape(3, 10, 2, 32, 40, 4, 4, 16, 4, 2)
    a = W.with_shared(W.place_contiguous(10, 2), [10, 11])
    b = W.with_shared(W.place_contiguous(10, 5), [10, 11])
    c = [[11, 3, 0, 10], [1, 2, 10, 11, 0], [4, 5, 6, 7, 8, 9, 3]]
    run_chain(sh, [a, b, c, a])


def test_matrix_larger_than_a_page_at_bench_width():
    """One layer of the mid-size shape's expert matrices (5.5 MiB each -> 6 MiB slabs),
    fewer experts: the copy kernels run their bulk path on arrivals."""
    sh = W.Shape(1, 12, 0, 2048, 1408, 16, 16, 128, 16, 2)
    run_chain(sh, [W.place_contiguous(12, 4), W.place_contiguous(12, 6)])


def test_failed_step_leaves_the_pool_unchanged():
    sh = W.Shape(1, 4, 0, 32, 32, 4, 4, 16, 4, 2)
    p0 = [[0, 1], [2, 3]]
    cur = [rand_bytes((60, r), n) for r, n in enumerate(dense_sizes(sh, p0))]
    with E.VmmPool(sh, p0) as pool:
        for r, a in enumerate(cur):
            pool.write(r, a)
        torch.cuda.synchronize()
        with pytest.raises(E.EmoeError) as ei:
            pool.reshard([[0, 1, 2]])          # expert 3 would be lost
        assert ei.value.code == 3
        assert pool.num_ranks() == 2
        assert all(np.array_equal(x, y) for x, y in zip(read_pool(pool, sh, p0), cur))


# ---- the store with slot tables: a step touches only the slots that change ---------------

def _read_slots(pool, sh):
    """{(rank, slot): bytes [L*3*m]} of every occupied slot."""
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    out = {}
    for r, table in enumerate(pool.tables()):
        for s, e in enumerate(table):
            if e >= 0:
                a = np.zeros(sh.n_layers * 3 * m, np.uint8)
                pool.read_slot(r, s, a)
                out[(r, s)] = a
    torch.cuda.synchronize()
    return out


def _slot_chain(sh, slots, steps, spare_slots, key=70):
    """Runs `steps` ([(want, cap_new), ...]) on a slot store and, in step with it, the oracle's
    in-place step on dense capacity-strided arenas; after every step each occupied slot must
    hold the oracle's bytes and the tables must agree."""
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    L3 = sh.n_layers * 3
    caps = [len(t) for t in slots]
    dense = [rand_bytes((key, r), L3 * c * m) for r, c in enumerate(caps)]
    torch.cuda.empty_cache()
    all_stats = []
    with E.VmmSlots(sh, slots, spare_slots=spare_slots) as pool:
        assert pool.tables() == slots
        for r, table in enumerate(slots):
            for s, e in enumerate(table):
                if e >= 0:
                    pool.write_slot(r, s, np.ascontiguousarray(dense[r].reshape(L3, caps[r], m)[:, s]).reshape(-1))
        torch.cuda.synchronize()
        for want, cap_new in steps:
            n_dev = max(len(slots), len(want))
            while len(dense) < n_dev:
                dense.append(rand_bytes((key + 1, len(dense)), L3 * cap_new[len(dense)] * m))
            spare_before = pool.info()["spare_slabs"]
            st = pool.reshard(want, cap_new)
            new_slots = oracle.reshard_experts_inplace(sh, slots, want, cap_new, dense[:n_dev])
            dense = dense[:len(want)]
            assert pool.tables() == new_slots
            arrivals = sum(1 for r, t in enumerate(new_slots) for s, e in enumerate(t)
                           if e >= 0 and not (r < len(slots) and slots[r][s] == e))
            kept = sum(1 for r, t in enumerate(new_slots) for s, e in enumerate(t)
                       if e >= 0 and r < len(slots) and slots[r][s] == e)
            left = sum(1 for r, t in enumerate(slots) for s, e in enumerate(t)
                       if e >= 0 and (r >= len(new_slots) or new_slots[r][s] != e))
            assert st["slabs_copied"] == arrivals * L3 and st["slabs_remapped"] == kept * L3
            assert st["bytes_copied"] == arrivals * L3 * m
            # pages are conserved: arrivals take from the spare list (or are created when it is
            # empty), experts that left give theirs back
            assert pool.info()["spare_slabs"] == max(spare_before - arrivals * L3, 0) + left * L3
            got = _read_slots(pool, sh)
            for (r, s), a in got.items():
                want_bytes = np.ascontiguousarray(dense[r].reshape(L3, len(new_slots[r]), m)[:, s]).reshape(-1)
                assert np.array_equal(a, want_bytes), (r, s)
            slots = new_slots
            all_stats.append(st)
    return all_stats


def test_slot_store_scale_up_down_and_reuse_of_spare_pages():
    sh = W.Shape(2, 12, 0, 64, 96, 4, 4, 16, 4, 2)
    slots = [[0, 1, 2, 3, 4, 5, -1, -1], [6, 7, 8, 9, 10, 11, -1, -1]]
    steps = [([[0, 1, 2], [6, 7, 8], [3, 4, 5], [9, 10, 11]], [8, 8, 4, 4]),          # 2 -> 4 devices
             ([[0, 1, 2, 9], [6, 7, 8, 3], [4, 5], [10, 11]], [8, 8, 4, 4]),          # experts swap devices
             ([[0, 1, 2, 9, 10, 11], [6, 7, 8, 3, 4, 5]], [8, 8]),                    # 4 -> 2 devices
             ([[0, 1, 2, 9, 10, 11], [6, 7, 8, 3, 4, 5]], [8, 8])]                    # nothing changes
    stats = _slot_chain(sh, slots, steps, spare_slots=6)
    assert stats[-1]["slabs_copied"] == 0 and stats[-1]["bytes_copied"] == 0
    assert stats[0]["alloc_ms"] == 0.0          # 6 arrivals, 6 spare slots: no page was created in the step


def test_slot_store_with_replicas_and_bench_width_matrices():
    sh = W.Shape(1, 8, 1, 2048, 1408, 16, 16, 128, 16, 2)       # 5.5 MiB matrices -> 6 MiB slabs
    slots = [[0, 1, 2, 3, 8, -1, -1], [4, 5, 6, 7, 8, -1, -1]]
    steps = [([[0, 1, 8, 4], [6, 7, 8], [2, 3, 5, 8, 0]], [7, 7, 6]),
             ([[0, 1, 2, 3, 8], [4, 5, 6, 7, 8]], [7, 7])]
    _slot_chain(sh, slots, steps, spare_slots=0)


def test_slot_store_refuses_a_step_before_touching_anything():
    sh = W.Shape(1, 4, 0, 32, 32, 4, 4, 16, 4, 2)
    slots = [[0, 1, -1], [2, 3, -1]]
    with E.VmmSlots(sh, slots, spare_slots=1) as pool:
        with pytest.raises(E.EmoeError) as ei:
            pool.reshard([[0, 2, 3], [1]], [3, 3])           # two arrivals, one free slot
        assert ei.value.code == 11
        with pytest.raises(E.EmoeError) as ei:
            pool.reshard([[0, 1], [2]], [3, 3])              # fine (3 leaves) ...
            pool.reshard([[0, 1, 3], [2]], [3, 3])           # ... but then nobody holds 3 any more
        assert ei.value.code == 3
        assert pool.tables() == [[0, 1, -1], [2, -1, -1]]
        assert pool.info()["spare_slabs"] == 3 + 3           # the spare slot's pages plus expert 3's
