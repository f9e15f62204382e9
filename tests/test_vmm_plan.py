"""Paged expert store, host side (no GPU): which slots a scale step keeps by re-mapping
and which it copies, against hand counts."""
from __future__ import annotations

import pytest

import paper_2510_02613_b200 as E
import workloads as W

MiB = 1 << 20


def shape(n_experts, layers=2, n_shared=0):
    return W.Shape(layers, n_experts - n_shared, n_shared, 64, 48, 4, 4, 16, 4, 2)   # m = 6144 B


def test_scale_up_ep4_to_ep6_keeps_what_stays_on_its_device():
    """The paper's scale-up scenario with 12 experts in contiguous ranges: device 0 keeps
    experts 0,1 of its 0,1,2; device 1 keeps 3 of its 3,4,5 (it now holds 2,3); devices 2
    and 3 hold ranges that lay on other devices before; devices 4,5 are new."""
    sh = shape(12)
    st = E.vmm_dry_run(sh, W.place_contiguous(12, 4), W.place_contiguous(12, 6), 2 * MiB)
    runs = 3 * sh.n_layers
    assert st["slabs_remapped"] == 3 * runs
    assert st["slabs_copied"] == 9 * runs
    assert st["bytes_copied"] == 9 * runs * 6144 == st["bytes_read"]
    assert st["physical_bytes"] == 12 * runs * 2 * MiB


def test_scale_down_ep4_to_ep2():
    """EP4 -> EP2: device 0 keeps its 0,1,2 and receives 3,4,5; device 1 (held 3,4,5)
    ends up with 6..11, none of which it had."""
    sh = shape(12)
    st = E.vmm_dry_run(sh, W.place_contiguous(12, 4), W.place_contiguous(12, 2), 2 * MiB)
    runs = 3 * sh.n_layers
    assert st["slabs_remapped"] == 3 * runs and st["slabs_copied"] == 9 * runs


def test_identity_step_copies_nothing_and_replicas_are_read_once():
    sh = shape(6)
    p = W.place_round_robin(6, 3)
    st = E.vmm_dry_run(sh, p, p, 2 * MiB)
    assert st["slabs_copied"] == 0 and st["bytes_copied"] == 0
    # expert 0 (old rank 0 only) arrives on ranks 1 and 2: two copies, one read
    st = E.vmm_dry_run(sh, p, [[0, 3], [1, 4, 0], [2, 5, 0]], 2 * MiB)
    runs = 3 * sh.n_layers
    assert st["slabs_remapped"] == 6 * runs and st["slabs_copied"] == 2 * runs
    assert st["bytes_copied"] == 2 * runs * 6144 and st["bytes_read"] == runs * 6144


def test_shared_experts_stay_where_a_rank_already_has_them():
    sh = shape(10, n_shared=2)
    old = W.with_shared(W.place_contiguous(8, 2), [8, 9])
    new = W.with_shared(W.place_contiguous(8, 4), [8, 9])
    st = E.vmm_dry_run(sh, old, new, 2 * MiB)
    runs = 3 * sh.n_layers
    # rank 0 keeps 0,1 + shared; rank 1 (held 4..7) now holds 2,3: keeps only its shared pair
    assert st["slabs_remapped"] == (4 + 2) * runs
    assert st["slabs_copied"] == (2 + 2 * 4) * runs


def test_dry_run_rejects_bad_input():
    sh = shape(4)
    with pytest.raises(E.EmoeError) as ei:
        E.vmm_dry_run(sh, [[0, 1], [2, 3]], [[0, 1, 2]], 2 * MiB)     # expert 3 lost
    assert ei.value.code == 3
    with pytest.raises(E.EmoeError) as ei:
        E.vmm_dry_run(sh, [[0, 1], [2, 3]], [[0, 1, 2, 3]], 1024)     # slab smaller than a matrix
    assert ei.value.code == 1
