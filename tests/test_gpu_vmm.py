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
