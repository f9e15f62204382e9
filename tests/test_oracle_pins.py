"""Pins of the CPU oracle against things that are not the oracle: numpy / torch
indexing of logical tensors, hand-written fixtures, identities and round trips.
A wrong offset formula, a swapped operand, a dropped loop or a wrong tie-break in
oracle/emoe_oracle.cpp fails at least one test here.  No GPU needed."""
from __future__ import annotations

import dataclasses
import os

import numpy as np
import pytest
import torch

import oracle
import workloads as W
from helpers import (FILL, attn_arenas, expert_arenas, kv_arenas, logical_attn, logical_experts,
                     logical_kv, rand_bytes)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def filled(sizes):
    return [np.full(n, FILL, dtype=np.uint8) for n in sizes]


def tiny_shape(**kw):
    base = dict(n_layers=3, n_routed=12, n_shared=0, d_model=8, d_ff=6, n_q_heads=8,
                n_kv_heads=4, head_dim=4, kv_block_tokens=4, elem_bytes=2)
    base.update(kw)
    return W.Shape(**base)


# ======================================================================== experts ======

PLACEMENTS = {
    "round_robin_2_4": (lambda: W.place_round_robin(12, 2), lambda: W.place_round_robin(12, 4)),
    "contig_4_6": (lambda: W.place_contiguous(12, 4), lambda: W.place_contiguous(12, 6)),
    "contig_4_2": (lambda: W.place_contiguous(12, 4), lambda: W.place_contiguous(12, 2)),
    "uneven_5_7": (lambda: W.place_contiguous(12, 5), lambda: W.place_contiguous(12, 7)),
    "scrambled": (lambda: [[5, 0, 11], [3, 9, 1, 7], [2, 10, 4, 8, 6]],
                  lambda: [[6, 5], [0, 1, 2, 3, 4], [11], [10, 9, 8, 7]]),
    "replicated_new": (lambda: W.place_contiguous(12, 3),
                       lambda: [[0, 1, 2, 11], [3, 4, 0, 5], [6, 7, 8], [9, 10, 11, 4]]),
}


@pytest.mark.parametrize("name", sorted(PLACEMENTS))
@pytest.mark.parametrize("elem_bytes", [1, 2, 4])
def test_experts_equal_numpy_gather_of_logical_tensor(name, elem_bytes):
    """Brute force: the new arena of rank r' is logical[:, :, P_new[r'], :]."""
    sh = tiny_shape(elem_bytes=elem_bytes)
    po, pn = (f() for f in PLACEMENTS[name])
    logical = logical_experts(sh)
    src = expert_arenas(logical, po)
    want = expert_arenas(logical, pn)
    dst = filled([a.size for a in want])
    oracle.reshard_experts(sh, po, pn, src, dst)
    for r, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % r


@pytest.mark.parametrize("name", sorted(PLACEMENTS))
def test_experts_fused_w13_equals_numpy_concatenate(name):
    """Fused gate|up layout: both sides built from the logical tensor with concatenate."""
    sh = tiny_shape()
    po, pn = (f() for f in PLACEMENTS[name])
    logical = logical_experts(sh)
    src = expert_arenas(logical, po, fused_w13=True)
    want = expert_arenas(logical, pn, fused_w13=True)
    assert [a.size for a in want] == oracle.expert_arena_bytes(sh, pn)
    dst = filled([a.size for a in want])
    oracle.reshard_experts(sh, po, pn, src, dst, fused_w13=True)
    for r, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % r
    # and it is a different byte order from the plain layout whenever a rank has > 1 slot
    plain = expert_arenas(logical, pn)
    assert any(not np.array_equal(a, b) for a, b in zip(plain, want) if a.size)


def test_experts_fused_w13_hand_written():
    """One layer, one rank with slots [A, B] -> two ranks [B], [A]; matrices of 2 bytes.
    Old arena: A.gate A.up B.gate B.up | A.down B.down."""
    sh = tiny_shape(n_layers=1, n_routed=2, d_model=1, d_ff=1, elem_bytes=2)
    src = [np.array([1, 1, 2, 2, 11, 11, 12, 12, 3, 3, 13, 13], np.uint8)]
    dst = filled([6, 6])
    oracle.reshard_experts(sh, [[0, 1]], [[1], [0]], src, dst, fused_w13=True)
    assert list(dst[0]) == [11, 11, 12, 12, 13, 13]       # B: gate up | down
    assert list(dst[1]) == [1, 1, 2, 2, 3, 3]             # A


def test_experts_shared_experts_on_every_rank():
    sh = tiny_shape(n_routed=10, n_shared=2)
    po = W.with_shared(W.place_contiguous(10, 2), [10, 11])
    pn = W.with_shared(W.place_contiguous(10, 3), [10, 11])
    logical = logical_experts(sh)
    dst = filled([a.size for a in expert_arenas(logical, pn)])
    oracle.reshard_experts(sh, po, pn, expert_arenas(logical, po), dst)
    for g, w in zip(dst, expert_arenas(logical, pn)):
        assert np.array_equal(g, w)


def test_experts_contiguous_equals_torch_cat_tensor_split():
    """Library special case: contiguous ranges -> cat along the slot axis, re-split."""
    sh = tiny_shape()
    po, pn = W.place_contiguous(12, 4), W.place_contiguous(12, 6)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    src = [rand_bytes((7, r), sh.n_layers * 3 * len(p) * m) for r, p in enumerate(po)]
    dst = filled([sh.n_layers * 3 * len(p) * m for p in pn])
    oracle.reshard_experts(sh, po, pn, src, dst)
    cat = torch.cat([torch.from_numpy(a).view(sh.n_layers, 3, len(p), m)
                     for a, p in zip(src, po)], dim=2)
    parts = cat.tensor_split(list(np.cumsum([len(p) for p in pn])[:-1]), dim=2)
    for g, w in zip(dst, parts):
        assert np.array_equal(g, w.contiguous().view(-1).numpy())


def test_experts_round_robin_equals_strided_slice():
    sh = tiny_shape()
    logical = logical_experts(sh)
    po, pn = W.place_round_robin(12, 2), W.place_round_robin(12, 4)
    dst = filled([sh.n_layers * 3 * len(p) * logical.shape[3] for p in pn])
    oracle.reshard_experts(sh, po, pn, expert_arenas(logical, po), dst)
    for r in range(4):
        assert np.array_equal(dst[r], np.ascontiguousarray(logical[:, :, r::4, :]).reshape(-1))


def test_experts_identity_is_memcpy_and_round_trip_is_identity():
    sh = tiny_shape()
    pa, pb = W.place_contiguous(12, 5), W.place_round_robin(12, 3)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    a0 = [rand_bytes((8, r), sh.n_layers * 3 * len(p) * m) for r, p in enumerate(pa)]
    same = filled([x.size for x in a0])
    oracle.reshard_experts(sh, pa, pa, a0, same)
    assert all(np.array_equal(x, y) for x, y in zip(a0, same))
    mid = filled([sh.n_layers * 3 * len(p) * m for p in pb])
    oracle.reshard_experts(sh, pa, pb, a0, mid)
    back = filled([x.size for x in a0])
    oracle.reshard_experts(sh, pb, pa, mid, back)
    assert all(np.array_equal(x, y) for x, y in zip(a0, back))


def test_experts_multiplicity_and_conservation():
    """Every expert lands exactly as often as the new placement lists it."""
    sh = tiny_shape(n_layers=1, d_model=4, d_ff=4, elem_bytes=1)
    m = 16
    po = W.place_contiguous(12, 3)
    pn = [[0, 1, 2, 11], [3, 4, 0, 5], [6, 7, 8], [9, 10, 11, 4]]
    logical = np.zeros((1, 3, 12, m), dtype=np.uint8)
    logical[:] = np.arange(12, dtype=np.uint8)[None, None, :, None]
    dst = filled([3 * len(p) * m for p in pn])
    oracle.reshard_experts(sh, po, pn, expert_arenas(logical, po), dst)
    hist = np.bincount(np.concatenate(dst), minlength=256)
    want = np.bincount([e for p in pn for e in p], minlength=12) * 3 * m
    assert np.array_equal(hist[:12], want) and hist[12:].sum() == 0
    assert sum(a.size for a in dst) == sum(len(p) for p in pn) * 3 * m


def test_experts_replica_choice_own_rank_first_then_smallest():
    """Hand-written: replicas with DIFFERENT contents pin which copy is read.
    old rank0 = [0, 1], old rank1 = [1, 2]; slabs are tagged 10*rank + slot + 1."""
    sh = tiny_shape(n_layers=1, n_routed=3, d_model=2, d_ff=2, elem_bytes=1)
    m = 4
    po = [[0, 1], [1, 2]]
    pn = [[1], [1], [1, 0, 2]]
    src = [np.repeat(np.array([[1, 2]] * 3, dtype=np.uint8).reshape(-1), m),
           np.repeat(np.array([[11, 12]] * 3, dtype=np.uint8).reshape(-1), m)]
    dst = filled([3 * len(p) * m for p in pn])
    oracle.reshard_experts(sh, po, pn, src, dst)
    assert set(dst[0]) == {2}          # new rank 0 keeps old rank 0's copy (slot 1)
    assert set(dst[1]) == {11}         # new rank 1 keeps old rank 1's copy (slot 0)
    assert list(dst[2][:3 * m:m]) == [2, 1, 12]   # no old rank 2: smallest (rank, slot)


@pytest.mark.parametrize("case,ep_new", [("up", 6), ("down", 2)])
def test_experts_paper_scenario_fixture(case, ep_new):
    """The paper's EP4 -> EP6 scale-up and EP4 -> EP2 scale-down, against a
    hand-written table of (new rank, new slot) <- (old rank, old slot)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_scale_ep4_ep6.txt"))
            if l.strip() and not l.startswith("#")]
    rows = [tuple(int(x) for x in r[1:]) for r in rows if r[0] == case]
    sh = tiny_shape(n_layers=2, d_model=2, d_ff=2, elem_bytes=2)
    m = 8
    po, pn = W.place_contiguous(12, 4), W.place_contiguous(12, ep_new)
    # every old slab (l, p, slot) of every rank carries its own tag
    src = []
    for r in range(4):
        a = np.zeros((2, 3, 3, m), dtype=np.uint8)
        for l in range(2):
            for p in range(3):
                for s in range(3):
                    a[l, p, s] = 1 + ((r * 3 + s) * 3 + p) * 2 + l
        src.append(a.reshape(-1))
    dst = filled([2 * 3 * len(p) * m for p in pn])
    oracle.reshard_experts(sh, po, pn, src, dst)
    assert len(rows) == 12
    for rn, sn, e, ro, so in rows:
        assert pn[rn][sn] == e and po[ro][so] == e
        got = dst[rn].reshape(2, 3, len(pn[rn]), m)
        for l in range(2):
            for p in range(3):
                assert set(got[l, p, sn]) == {1 + ((ro * 3 + so) * 3 + p) * 2 + l}


def test_experts_missing_source_is_an_error():
    sh = tiny_shape(n_layers=1, n_routed=3, d_model=2, d_ff=2)
    with pytest.raises(ValueError):
        oracle.reshard_experts(sh, [[0, 1]], [[0, 2]], [np.zeros(48, np.uint8)],
                               [np.zeros(48, np.uint8)])


# ====================================================================== attention ======

@pytest.mark.parametrize("c,d", [(1, 2), (2, 4), (4, 1), (2, 2), (4, 2), (1, 4)])
@pytest.mark.parametrize("elem_bytes", [2, 4])
def test_attn_equals_numpy_split_of_logical_matrices(c, d, elem_bytes):
    sh = tiny_shape(elem_bytes=elem_bytes)
    logical = logical_attn(sh)
    src, want = attn_arenas(logical, c), attn_arenas(logical, d)
    dst = filled([a.size for a in want])
    oracle.reshard_attn(sh, c, d, src, dst)
    for t, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % t


def test_attn_gqa_shapes_and_torch_cat_chunk():
    """Library special case on one layer: cat(shards, dim).chunk(d, dim) with dim 0
    for q/k/v and dim 1 for o, for a GQA shape (Hq != Hkv)."""
    sh = tiny_shape(n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=4, d_model=6)
    c, d = 1, 2
    D, b = sh.d_model, sh.elem_bytes
    q, kv = sh.n_q_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
    src = [rand_bytes(11, (2 * q * D + 2 * kv * D) * b)]
    t = torch.from_numpy(src[0])
    sizes = [q * D * b, kv * D * b, kv * D * b, D * q * b]
    Q, K, V, O = t.split(sizes)
    Q, K, V = Q.view(q, D * b), K.view(kv, D * b), V.view(kv, D * b)
    O = O.view(D, q, b)
    dst = filled(oracle.attn_arena_bytes(sh, d))
    oracle.reshard_attn(sh, c, d, src, dst)
    for r in range(d):
        want = torch.cat([Q.chunk(d, 0)[r].reshape(-1), K.chunk(d, 0)[r].reshape(-1),
                          V.chunk(d, 0)[r].reshape(-1), O.chunk(d, 1)[r].reshape(-1)])
        assert np.array_equal(dst[r], want.numpy())


def test_attn_fixed_tp_is_memcpy_and_round_trip():
    sh = tiny_shape()
    a0 = [rand_bytes((12, t), n) for t, n in enumerate(oracle.attn_arena_bytes(sh, 2))]
    same = filled([a.size for a in a0])
    oracle.reshard_attn(sh, 2, 2, a0, same)      # the paper's fixed-TP case (Sec. 5.2)
    assert all(np.array_equal(x, y) for x, y in zip(a0, same))
    mid = filled(oracle.attn_arena_bytes(sh, 4))
    oracle.reshard_attn(sh, 2, 4, a0, mid)
    back = filled([a.size for a in a0])
    oracle.reshard_attn(sh, 4, 2, mid, back)
    assert all(np.array_equal(x, y) for x, y in zip(a0, back))


def test_attn_rejects_tp_not_dividing_heads():
    sh = tiny_shape(n_kv_heads=2, n_q_heads=12)
    with pytest.raises(ValueError):      # 3 ranks: neither 2 % 3 nor 3 % 2 is zero
        oracle.reshard_attn(sh, 1, 3, [np.zeros(oracle.attn_arena_bytes(sh, 1)[0], np.uint8)],
                            [np.zeros(1, np.uint8)] * 3)


@pytest.mark.parametrize("c,d", [(1, 4), (2, 8), (8, 2), (4, 8), (8, 4), (8, 8), (2, 4)])
def test_attn_more_ranks_than_kv_heads_equals_numpy_head_slices(c, d):
    """Hkv = 2: with TP > 2 every rank holds ONE k/v head (head floor(t*Hkv/T)), q and o
    are still split T ways.  Expected arenas are numpy slices of the logical matrices."""
    sh = tiny_shape(n_q_heads=8, n_kv_heads=2)
    logical = logical_attn(sh)
    src = attn_arenas(logical, c, sh.head_dim)
    want = attn_arenas(logical, d, sh.head_dim)
    assert [a.size for a in want] == oracle.attn_arena_bytes(sh, d)
    dst = filled([a.size for a in want])
    oracle.reshard_attn(sh, c, d, src, dst)
    for t, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % t


# ============================================================================= KV ======

def kv_cfgs(sh, c, d, seq_lens, nb_old, nb_new, seed=5, new_order="random"):
    B = sh.kv_block_tokens
    bo = W.make_block_table(W.rng.stream_key(seed, 1), seq_lens, B, nb_old)
    bn = W.make_block_table(W.rng.stream_key(seed, 2), seq_lens, B, nb_new, order=new_order)
    return (W.ParallelConfig(1, c, [[]], nb_old, seq_lens, bo),
            W.ParallelConfig(1, d, [[]], nb_new, seq_lens, bn))


@pytest.mark.parametrize("c,d", [(1, 2), (2, 4), (4, 2), (1, 1), (2, 2), (4, 1)])
def test_kv_equals_numpy_scatter_of_logical_cache(c, d):
    """Tokens keep sequence, position and head identity: both layouts are
    scatters of the same logical [L,2,block,B,Hkv,hd] cache through the tables."""
    sh = tiny_shape()
    old, new = kv_cfgs(sh, c, d, [9, 4, 13, 1], 11, 14)
    logical = logical_kv(sh, old)
    src = kv_arenas(logical, sh, old)
    want = kv_arenas(logical, sh, new)          # unmapped blocks keep the 0xCD fill
    dst = filled([a.size for a in want])
    oracle.reshard_kv(sh, old, new, src, dst)
    for t, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % t


@pytest.mark.parametrize("c,d", [(1, 8), (2, 8), (8, 2), (4, 8), (8, 4), (8, 16), (16, 1)])
def test_kv_more_ranks_than_heads_equals_numpy_scatter(c, d):
    """Hkv = 4 and up to 16 ranks: a rank beyond the head count holds one (replicated)
    head; both layouts are scatters of the same logical cache."""
    sh = tiny_shape(n_q_heads=16, n_kv_heads=4)
    old, new = kv_cfgs(sh, c, d, [9, 4, 13, 1], 11, 14)
    logical = logical_kv(sh, old)
    src = kv_arenas(logical, sh, old)
    want = kv_arenas(logical, sh, new)
    assert [a.size for a in want] == oracle.kv_arena_bytes(sh, d, 14)
    dst = filled([a.size for a in want])
    oracle.reshard_kv(sh, old, new, src, dst)
    for t, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % t


@pytest.mark.parametrize("c,d", [(1, 2), (2, 4), (4, 2), (2, 2), (4, 1), (2, 8), (8, 4)])
def test_kv_head_major_equals_numpy_swapaxes(c, d):
    """Head-major blocks: both layouts are the token-major pools with the token and head
    axes swapped (numpy), so tokens still keep sequence, position and head identity."""
    sh = tiny_shape(n_q_heads=8, n_kv_heads=4)
    old, new = kv_cfgs(sh, c, d, [9, 4, 13, 1], 11, 14)
    logical = logical_kv(sh, old)
    src = kv_arenas(logical, sh, old, head_major=True)
    want = kv_arenas(logical, sh, new, head_major=True)
    dst = filled([a.size for a in want])
    oracle.reshard_kv(sh, old, new, src, dst, head_major=True)
    for t, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % t


def test_kv_head_major_hand_written():
    """The two-head example of the token-major test, blocks stored head-major: old block
    1 holds h0t0 h0t1 h1t0 h1t1."""
    sh = tiny_shape(n_layers=1, n_kv_heads=2, head_dim=1, kv_block_tokens=2, elem_bytes=2)
    old = W.ParallelConfig(1, 1, [[]], 2, [2], np.array([[1]], np.int32))
    new = W.ParallelConfig(1, 2, [[]], 1, [2], np.array([[0]], np.int32))
    K = [0] * 8 + [1, 2, 5, 6, 3, 4, 7, 8]
    V = [0] * 8 + [21, 22, 25, 26, 23, 24, 27, 28]
    dst = filled([8, 8])
    oracle.reshard_kv(sh, old, new, [np.array(K + V, dtype=np.uint8)], dst, head_major=True)
    assert list(dst[0]) == [1, 2, 5, 6, 21, 22, 25, 26]      # head 0: K t0,t1 then V t0,t1
    assert list(dst[1]) == [3, 4, 7, 8, 23, 24, 27, 28]      # head 1


def test_kv_replicated_head_source_is_own_rank_then_smallest():
    """Hand-written: one KV head, TP2 -> TP3, the two old replicas hold DIFFERENT bytes
    (1s and 2s).  New rank 0 keeps old rank 0's, new rank 1 old rank 1's, new rank 2 (no
    old rank 2) takes the smallest holder's, old rank 0."""
    sh = tiny_shape(n_layers=1, n_q_heads=6, n_kv_heads=1, head_dim=1, kv_block_tokens=2,
                    elem_bytes=1)
    bt = np.array([[0]], np.int32)
    old = W.ParallelConfig(1, 2, [[]], 1, [2], bt)
    new = W.ParallelConfig(1, 3, [[]], 1, [2], bt)
    src = [np.full(4, 1, np.uint8), np.full(4, 2, np.uint8)]       # [K|V][1 block][2 tok][1 head][1 B]
    dst = filled([4, 4, 4])
    oracle.reshard_kv(sh, old, new, src, dst)
    assert [set(a) for a in dst] == [{1}, {2}, {1}]
    # and the k / v weights follow the same rule (q and o rows are filled with 9s)
    D = sh.d_model
    def attn_arena(tag, tp):
        q = sh.n_q_heads // tp * D
        return np.concatenate([np.full(q, 9, np.uint8), np.full(2 * D, tag, np.uint8),
                               np.full(q, 9, np.uint8)])
    a_dst = filled(oracle.attn_arena_bytes(sh, 3))
    oracle.reshard_attn(sh, 2, 3, [attn_arena(1, 2), attn_arena(2, 2)], a_dst)
    q3 = sh.n_q_heads // 3 * D
    assert [set(a[q3:q3 + 2 * D]) for a in a_dst] == [{1}, {2}, {1}]


def test_kv_same_table_same_tp_leaves_mapped_blocks_unchanged():
    """The paper's case (fixed TP, cache reused as is): output == input on every
    mapped block, and nothing else is written."""
    sh = tiny_shape()
    old, _ = kv_cfgs(sh, 2, 2, [9, 4, 13], 9, 9)
    src = [rand_bytes((13, t), n) for t, n in enumerate(oracle.kv_arena_bytes(sh, 2, 9))]
    dst = filled([a.size for a in src])
    oracle.reshard_kv(sh, old, old, src, dst)
    used = sorted(int(x) for x in old.block_table.reshape(-1) if x >= 0)
    free = [p for p in range(9) if p not in used]
    for s, g in zip(src, dst):
        s6 = s.reshape(sh.n_layers, 2, 9, -1)
        g6 = g.reshape(sh.n_layers, 2, 9, -1)
        assert np.array_equal(g6[:, :, used], s6[:, :, used])
        assert (g6[:, :, free] == FILL).all()


def test_kv_round_trip_and_byte_conservation():
    sh = tiny_shape()
    old, new = kv_cfgs(sh, 2, 4, [16, 7, 5], 8, 10)
    logical = logical_kv(sh, old)
    src = kv_arenas(logical, sh, old)
    mid = filled(oracle.kv_arena_bytes(sh, 4, 10))
    oracle.reshard_kv(sh, old, new, src, mid)
    back = filled([a.size for a in src])
    oracle.reshard_kv(sh, new, old, mid, back)
    assert all(np.array_equal(x, y) for x, y in zip(src, back))
    n_blocks = sum(-(-n // sh.kv_block_tokens) for n in old.seq_lens)
    moved = sum(int((a != FILL).sum()) for a in mid)
    total = (sh.n_layers * 2 * n_blocks * sh.kv_block_tokens * sh.n_kv_heads * sh.head_dim
             * sh.elem_bytes)
    # random payload bytes equal the fill value now and then: bound, not equality
    assert total * 0.98 <= moved <= total


def test_kv_hand_written_two_heads_split():
    """One layer, one block of 2 tokens, 2 heads of 1 two-byte element, TP1 -> TP2,
    old physical block 1 of 2, new physical block 0 of 1: written out by hand."""
    sh = tiny_shape(n_layers=1, n_kv_heads=2, head_dim=1, kv_block_tokens=2, elem_bytes=2)
    old = W.ParallelConfig(1, 1, [[]], 2, [2], np.array([[1]], np.int32))
    new = W.ParallelConfig(1, 2, [[]], 1, [2], np.array([[0]], np.int32))
    # old arena: [K|V][block 0, block 1][tok][head][2 bytes]
    K = [0, 0, 0, 0, 0, 0, 0, 0, 1, 2, 3, 4, 5, 6, 7, 8]        # block 1: t0h0 t0h1 t1h0 t1h1
    V = [0, 0, 0, 0, 0, 0, 0, 0, 21, 22, 23, 24, 25, 26, 27, 28]
    src = [np.array(K + V, dtype=np.uint8)]
    dst = filled([8, 8])
    oracle.reshard_kv(sh, old, new, src, dst)
    assert list(dst[0]) == [1, 2, 5, 6, 21, 22, 25, 26]      # head 0: K t0,t1 then V t0,t1
    assert list(dst[1]) == [3, 4, 7, 8, 23, 24, 27, 28]      # head 1


# ===================================================================== arena sizes =====

def test_arena_sizes_match_numpy_shapes():
    sh = tiny_shape()
    logical = logical_experts(sh)
    pl = W.place_contiguous(12, 5)
    assert oracle.expert_arena_bytes(sh, pl) == [a.size for a in expert_arenas(logical, pl)]
    assert oracle.attn_arena_bytes(sh, 2) == [a.size for a in attn_arenas(logical_attn(sh), 2)]
    old, _ = kv_cfgs(sh, 2, 2, [9, 4], 6, 6)
    assert oracle.kv_arena_bytes(sh, 2, 6) == [a.size for a in
                                               kv_arenas(logical_kv(sh, old), sh, old)]


def test_published_step_bytes_of_the_five_configs():
    """Whole-step byte counts of C1..C4, computed independently from the shapes."""
    want = {"c1_tiny": 31457280, "c2_mid": 32161923072, "c3_fine": 56509857792,
            "c4_large": 25434259456}
    for name, total in want.items():
        wl = W.make_workload(name)
        sh = wl.shape
        used = sum(-(-n // sh.kv_block_tokens) for n in wl.old.seq_lens)
        kv_moved = (sh.n_layers * 2 * used * sh.kv_block_tokens * sh.n_kv_heads * sh.head_dim
                    * sh.elem_bytes)
        got = (sum(oracle.expert_arena_bytes(sh, wl.new.placement))
               + sum(oracle.attn_arena_bytes(sh, wl.new.tp)) + kv_moved)
        assert got == total, name


# ============================================================ in-place expert step ======

def slot_arenas(logical, slots, key):
    """Arena [L, 3, cap, m] of every rank: occupied slots hold their expert's logical
    matrices (numpy indexing), free slots hold bytes of their own (so that a write to a
    slot that must stay untouched is seen)."""
    L, _, _, m = logical.shape
    out = []
    for r, table in enumerate(slots):
        a = rand_bytes((key, r), L * 3 * len(table) * m).reshape(L, 3, len(table), m).copy()
        for s, e in enumerate(table):
            if e >= 0:
                a[:, :, s] = logical[:, :, e]
        out.append(a.reshape(-1))
    return out


INPLACE_CASES = {
    # old slot tables, wanted experts per new rank, capacity of the new ranks
    "grow_2_3": ([[0, 1, 2, -1, -1], [3, 4, 5, -1, -1]], [[0, 1], [3, 4], [2, 5]], [5, 5, 3]),
    "grow_with_swaps": ([[0, 1, 2, -1, -1, -1], [3, 4, 5, -1, -1, -1]],
                        [[5, 0, 4], [1, 3], [2, 0, 3]], [6, 6, 4]),
    "shrink_3_2": ([[0, 1, -1, -1], [2, 3, -1, -1], [4, 5, -1]], [[0, 1, 4, 2], [3, 5, 2]], [4, 4]),
    "holes_first": ([[-1, 0, -1, 1], [-1, -1, 2, 3]], [[3, 2, 0], [1, 3]], [4, 4]),
    "replicated": ([[0, 1, -1, -1], [1, 2, -1, -1]], [[0, 2, 1], [0, 1], [1, 2, 0]], [4, 4, 3]),
    "nothing_moves": ([[0, 1, -1], [2, -1, 3]], [[1, 0], [3, 2]], [3, 3]),
}


@pytest.mark.parametrize("name", sorted(INPLACE_CASES))
def test_inplace_step_against_numpy_indexing_of_the_logical_tensor(name):
    """After the step every occupied slot of every rank holds logical[:, :, expert]; a kept
    expert is in the slot it had; every other byte - free slots, slots of experts that
    left - is exactly what it was."""
    old, want, cap_new = INPLACE_CASES[name]
    n_exp = 1 + max(e for t in old for e in t)
    sh = tiny_shape(n_routed=n_exp, n_layers=2)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    logical = logical_experts(sh, key=11)
    arenas = slot_arenas(logical, old, 12)
    for r in range(len(old), len(want)):          # added devices: fresh arenas
        arenas.append(rand_bytes((13, r), sh.n_layers * 3 * cap_new[r] * m))
    before = [a.copy() for a in arenas]
    new = oracle.reshard_experts_inplace(sh, old, want, cap_new, arenas)
    assert len(new) == len(want)
    for r, table in enumerate(new):
        assert len(table) == cap_new[r]
        assert sorted(e for e in table if e >= 0) == sorted(want[r])
        got = arenas[r].reshape(sh.n_layers, 3, cap_new[r], m)
        was = before[r].reshape(sh.n_layers, 3, cap_new[r], m)
        for s, e in enumerate(table):
            if e >= 0:
                assert np.array_equal(got[:, :, s], logical[:, :, e]), (r, s, e)
                if r < len(old) and e in old[r]:
                    assert old[r][s] == e                       # kept where it was
                else:
                    assert r >= len(old) or old[r][s] == -1     # arrivals use old-free slots only
            else:
                assert np.array_equal(got[:, :, s], was[:, :, s]), (r, s)   # untouched
    for r in range(len(want), len(old)):          # removed devices are not written
        assert np.array_equal(arenas[r], before[r])


def test_inplace_arrivals_take_lowest_free_slots_in_listed_order():
    old = [[7, -1, 3, -1, -1]]
    # 9 and 8 have no source here; the table itself does not need one
    assert oracle.inplace_slots(old, [[3, 9, 8]], [5]) == [[-1, 9, 3, 8, -1]]
    assert oracle.inplace_slots(old, [[8, 9, 3]], [5]) == [[-1, 8, 3, 9, -1]]
    assert oracle.inplace_slots(old, [[7, 3]], [5]) == old
    assert oracle.inplace_slots(old, [[]], [5]) == [[-1] * 5]


def test_inplace_refuses_what_the_capacity_cannot_hold():
    with pytest.raises(ValueError, match="free slots"):
        oracle.inplace_slots([[0, 1, -1]], [[2, 3]], [3])      # one free slot, two arrivals
    with pytest.raises(ValueError, match="capacity"):
        oracle.inplace_slots([[0, 1, -1]], [[0]], [4])         # a staying rank cannot grow
    with pytest.raises(ValueError, match="twice"):
        oracle.inplace_slots([[0, 1, -1]], [[0, 0]], [3])
    sh = tiny_shape(n_routed=3, n_layers=1)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    with pytest.raises(ValueError, match="no copy"):
        oracle.reshard_experts_inplace(sh, [[0, -1]], [[0, 2]], [2], [np.zeros(3 * 2 * m, np.uint8)])


def test_inplace_source_is_the_smallest_rank_and_slot():
    """Replicas with different contents: the arrival must carry the bytes of the smallest
    (rank, slot) that held the expert before the step."""
    sh = tiny_shape(n_layers=1, n_routed=2, d_model=2, d_ff=2, elem_bytes=1)
    m = 4
    old = [[-1, 1, 0], [1, -1, -1]]
    tag = lambda r, s: 10 * r + s + 1
    arenas = [np.repeat(np.array([[tag(r, s) for s in range(3)]] * 3, np.uint8).reshape(-1), m)
              for r in range(2)]
    arenas.append(np.zeros(3 * 2 * m, np.uint8))
    new = oracle.reshard_experts_inplace(sh, old, [[0, 1], [1, 0], [1, 0]], [3, 3, 2], arenas)
    assert new == [[-1, 1, 0], [1, 0, -1], [1, 0]]
    a1 = arenas[1].reshape(3, 3, m)
    assert set(a1[:, 1].reshape(-1)) == {tag(0, 2)}          # expert 0 came from rank 0 slot 2
    a2 = arenas[2].reshape(3, 2, m)
    assert set(a2[:, 0].reshape(-1)) == {tag(0, 1)}          # expert 1: rank 0 slot 1, not rank 1 slot 0
    assert set(a2[:, 1].reshape(-1)) == {tag(0, 2)}


def test_inplace_chain_reuses_slots_freed_by_the_previous_step():
    """A slot freed in one step is available to arrivals of the NEXT step; compacted to the
    wanted order, every step agrees with the out-of-place expert re-pack."""
    sh = tiny_shape(n_routed=8, n_layers=2)
    m = sh.d_model * sh.d_ff * sh.elem_bytes
    logical = logical_experts(sh, key=21)
    slots = [[0, 1, 2, 3, -1, -1], [4, 5, 6, 7, -1, -1]]
    arenas = slot_arenas(logical, slots, 22)
    steps = [([[0, 1, 4, 5], [6, 7, 2, 3]], [6, 6]),           # two arrivals each way
             ([[0, 1, 4, 5, 3], [6, 7, 2]], [6, 6]),           # 3 comes back into a slot freed before
             ([[0, 1], [6, 7], [2, 3, 4, 5]], [6, 6, 4]),      # grow
             ([[0, 1, 2, 3, 4, 5], [6, 7]], [6, 6])]           # shrink again
    for want, cap in steps:
        while len(arenas) < len(want):
            arenas.append(rand_bytes((23, len(arenas)), sh.n_layers * 3 * cap[len(arenas)] * m))
        slots = oracle.reshard_experts_inplace(sh, slots, want, cap, arenas[:max(len(slots), len(want))])
        arenas = arenas[:len(want)]
        for r, table in enumerate(slots):
            got = arenas[r].reshape(sh.n_layers, 3, len(table), m)
            order = [table.index(e) for e in want[r]]
            compact = np.ascontiguousarray(got[:, :, order]).reshape(-1)
            assert np.array_equal(compact, expert_arenas(logical, [want[r]])[0])
    assert slots == [[0, 1, 2, 3, 4, 5], [-1, -1, 6, 7, -1, -1]]      # worked out by hand


@pytest.mark.parametrize("case", ["up", "down"])
def test_inplace_paper_scenario_fixture(case):
    """The paper's scale-up / scale-down scenario in its in-place form against hand-written
    slot tables and a hand-written list of the only transfers the step may make."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_scale_inplace.txt"))
            if l.strip() and not l.startswith("#")]
    want_slots = {int(r[2]): [int(x) for x in r[3:]] for r in rows if r[0] == "slots" and r[1] == case}
    copies = [tuple(int(x) for x in r[2:]) for r in rows if r[0] == "copy" and r[1] == case]
    if case == "up":
        old = [[3 * r, 3 * r + 1, 3 * r + 2, -1] for r in range(4)]
        want, cap = [[0, 1], [3, 2], [6, 5], [9, 8], [4, 7, 1], [10, 11]], [4] * 6
    else:
        old = [[0, 1, -1, -1], [3, -1, -1, 2], [6, 7, -1, 5], [9, 10, 11, 8]]
        want, cap = [[0, 1, 6, 7], [3, 2, 9, 5]], [4, 4]
    sh = tiny_shape(n_layers=2, d_model=2, d_ff=2, elem_bytes=2)
    m = 8
    n_dev = max(len(old), len(want))
    tag = lambda r, s, l, p: 1 + ((r * 4 + s) * 3 + p) * 2 + l      # every slab its own byte value
    arenas = []
    for r in range(n_dev):
        a = np.zeros((2, 3, 4, m), np.uint8)
        for l in range(2):
            for p in range(3):
                for s in range(4):
                    a[l, p, s] = tag(r, s, l, p)
        arenas.append(a.reshape(-1))
    new = oracle.reshard_experts_inplace(sh, old, want, cap, arenas)
    assert new == [want_slots[r] for r in range(len(want))]
    written = {(rn, sn): (ro, so) for rn, sn, e, ro, so in copies}
    for rn, sn, e, ro, so in copies:
        assert new[rn][sn] == e and old[ro][so] == e
    for r in range(n_dev):
        got = arenas[r].reshape(2, 3, 4, m)
        for s in range(4):
            ro, so = written.get((r, s), (r, s))                  # everything else is untouched
            for l in range(2):
                for p in range(3):
                    assert set(got[l, p, s]) == {tag(ro, so, l, p)}, (r, s)


# ================================================================= fused qkv ===========

from helpers import attn_arenas_fused_qkv  # noqa: E402


@pytest.mark.parametrize("hq,hkv,c,d", [(8, 4, 1, 2), (8, 4, 4, 2), (8, 8, 2, 4), (8, 2, 1, 2),
                                        (8, 2, 2, 4), (8, 2, 8, 2), (8, 2, 4, 8), (16, 4, 2, 2)])
@pytest.mark.parametrize("elem_bytes", [1, 2])
def test_attn_fused_qkv_equals_numpy_concatenate_of_head_slices(hq, hkv, c, d, elem_bytes):
    sh = tiny_shape(n_q_heads=hq, n_kv_heads=hkv, head_dim=3, d_model=5, elem_bytes=elem_bytes, n_layers=2)
    logical = logical_attn(sh)
    src = attn_arenas_fused_qkv(logical, c, hq, hkv, sh.head_dim)
    want = attn_arenas_fused_qkv(logical, d, hq, hkv, sh.head_dim)
    assert [a.size for a in want] == oracle.attn_arena_bytes(sh, d)
    dst = filled([a.size for a in want])
    oracle.reshard_attn(sh, c, d, src, dst, fused_qkv=True)
    for r, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % r


def test_attn_fused_qkv_hand_written():
    """4 query heads, 2 KV heads, head_dim 1, d_model 1, one byte per element, one layer.
    Logical rows tagged q: 10..13, k: 20,21, v: 30,31, o (one row of 4 columns): 40..43.
    TP1 arena: [q0 q1 k0 v0 | q2 q3 k1 v1 | o0 o1 o2 o3];
    TP2 arenas: rank 0 [q0 q1 k0 v0 | o0 o1], rank 1 [q2 q3 k1 v1 | o2 o3];
    TP4 arenas: rank t [q_t k_(t//2) v_(t//2) | o_t]."""
    sh = tiny_shape(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=1, d_model=1, elem_bytes=1)
    tp1 = [np.array([10, 11, 20, 30, 12, 13, 21, 31, 40, 41, 42, 43], np.uint8)]
    tp2 = [np.array([10, 11, 20, 30, 40, 41], np.uint8), np.array([12, 13, 21, 31, 42, 43], np.uint8)]
    tp4 = [np.array([10, 20, 30, 40], np.uint8), np.array([11, 20, 30, 41], np.uint8),
           np.array([12, 21, 31, 42], np.uint8), np.array([13, 21, 31, 43], np.uint8)]
    for a, b in ((tp1, tp2), (tp2, tp1), (tp1, tp4), (tp4, tp2), (tp2, tp4), (tp4, tp1)):
        dst = filled([x.size for x in b])
        oracle.reshard_attn(sh, len(a), len(b), a, dst, fused_qkv=True)
        assert all(np.array_equal(g, w) for g, w in zip(dst, b)), (len(a), len(b))


def test_attn_fused_qkv_with_one_query_head_per_kv_head_interleaves_q_k_v():
    """Hq == Hkv: the fused matrix is [q0 k0 v0 q1 k1 v1 ...]; un-fusing it with a numpy
    reshape gives the plain q | k | v pieces."""
    sh = tiny_shape(n_q_heads=4, n_kv_heads=4, head_dim=2, d_model=3, elem_bytes=2, n_layers=2)
    logical = logical_attn(sh)
    fused = attn_arenas_fused_qkv(logical, 2, 4, 4, 2)
    plain = attn_arenas(logical, 2)
    row = 3 * 2
    for f, p in zip(fused, plain):
        f = f.reshape(2, -1)
        p = p.reshape(2, -1)
        n_qkv = 3 * 2 * 2 * row                                   # 2 heads per rank, q k v, hd rows
        x = f[:, :n_qkv].reshape(2, 2, 3, 2 * row)                # [layer, head, q|k|v, head bytes]
        unfused = np.concatenate([x[:, :, 0].reshape(2, -1), x[:, :, 1].reshape(2, -1),
                                  x[:, :, 2].reshape(2, -1)], axis=1)
        assert np.array_equal(unfused, p[:, :n_qkv])
        assert np.array_equal(f[:, n_qkv:], p[:, n_qkv:])          # o is the same


def test_attn_fused_qkv_rejects_query_heads_not_divisible_by_kv_heads():
    sh = tiny_shape(n_q_heads=6, n_kv_heads=4, head_dim=2)
    with pytest.raises(ValueError):
        oracle.reshard_attn(sh, 1, 2, [np.zeros(oracle.attn_arena_bytes(sh, 1)[0], np.uint8)],
                            filled(oracle.attn_arena_bytes(sh, 2)), fused_qkv=True)


# ==================================================== experts with scale tensors =======

def scaled_arenas(weights, scales, placement):
    """Arena of a rank = its experts' weights [L,3,n,m] flattened, zero padding up to a
    multiple of 256 bytes, then their scales [L,3,n,ms] flattened (numpy.concatenate)."""
    out = []
    for p in placement:
        w = np.ascontiguousarray(weights[:, :, list(p)]).reshape(-1)
        pad = np.zeros(-w.size % 256, np.uint8)
        out.append(np.concatenate([w, pad, np.ascontiguousarray(scales[:, :, list(p)]).reshape(-1)]))
    return out


@pytest.mark.parametrize("name", sorted(PLACEMENTS))
@pytest.mark.parametrize("ms", [4, 24])
def test_experts_with_scales_equal_numpy_gather_of_both_logical_tensors(name, ms):
    sh = dataclasses.replace(tiny_shape(elem_bytes=1, d_model=9, d_ff=7), expert_scale_bytes=ms)
    po, pn = (f() for f in PLACEMENTS[name])
    weights = logical_experts(sh, key=41)
    scales = rand_bytes(42, sh.n_layers * 3 * sh.n_experts * ms).reshape(sh.n_layers, 3, sh.n_experts, ms)
    src = scaled_arenas(weights, scales, po)
    want = scaled_arenas(weights, scales, pn)
    assert [a.size for a in want] == oracle.expert_arena_bytes(sh, pn)
    dst = [np.zeros(a.size, np.uint8) for a in want]       # padding is written by nobody: stays zero
    oracle.reshard_experts(sh, po, pn, src, dst)
    for r, (g, w) in enumerate(zip(dst, want)):
        assert np.array_equal(g, w), "rank %d" % r
        assert oracle.expert_scale_base(sh, len(pn[r])) % 256 == 0


def test_experts_with_scales_hand_written():
    """One layer, matrices of 2 bytes, scales of 1 byte.  Rank with 2 experts: weights
    occupy 3*2*2 = 12 bytes, scales start at byte 256."""
    sh = dataclasses.replace(tiny_shape(n_layers=1, n_routed=2, d_model=1, d_ff=1, elem_bytes=2),
                             expert_scale_bytes=1)
    old = np.zeros(256 + 6, np.uint8)
    old[:12] = [1, 1, 2, 2, 3, 3, 4, 4, 5, 5, 6, 6]       # gate e0,e1 | up e0,e1 | down e0,e1
    old[256:262] = [11, 12, 13, 14, 15, 16]
    dst = [np.zeros(256 + 3, np.uint8), np.zeros(256 + 3, np.uint8)]
    oracle.reshard_experts(sh, [[0, 1]], [[1], [0]], [old], dst)
    assert list(dst[0][:6]) == [2, 2, 4, 4, 6, 6] and list(dst[0][256:]) == [12, 14, 16]
    assert list(dst[1][:6]) == [1, 1, 3, 3, 5, 5] and list(dst[1][256:]) == [11, 13, 15]
    assert not dst[0][6:256].any() and not dst[1][6:256].any()


# ============================================================ compacting block table ===

def test_compact_block_table_hand_written_and_properties():
    """Two sequences of 5 and 3 tokens in 2-token blocks need 3 + 2 blocks; in a pool of 8
    with blocks 1 and 4 taken they get 0, 2, 3 and 5, 6 (written by hand)."""
    t = oracle.compact_block_table([5, 3], 2, 8, in_use=[1, 4])
    assert t.tolist() == [[0, 2, 3], [5, 6, -1]]
    assert oracle.compact_block_table([5, 3], 2, 5).tolist() == [[0, 1, 2], [3, 4, -1]]   # fresh pool: identity
    rng = np.random.default_rng(3)
    for _ in range(20):
        nb = int(rng.integers(6, 30))
        in_use = [int(x) for x in rng.permutation(nb)[:int(rng.integers(0, nb // 2))]]
        free = sorted(set(range(nb)) - set(in_use))
        lens = [int(x) for x in rng.integers(0, 8, size=3)]
        if sum(-(-n // 3) for n in lens) > len(free):
            continue
        flat = [int(x) for row in oracle.compact_block_table(lens, 3, nb, in_use) for x in row if x >= 0]
        assert flat == free[:len(flat)]


# ======================================================= attention for added replicas ===

@pytest.mark.parametrize("c,d,replicas", [(2, 2, 3), (1, 2, 2), (4, 2, 2)])
def test_attn_replicas_each_equal_the_numpy_split(c, d, replicas):
    """Provisioning added data-parallel replicas: every replica's shard t is the numpy split of
    the logical matrices, whatever the old TP degree; a dropped or misplaced replica shows."""
    sh = tiny_shape(n_layers=2)
    logical = logical_attn(sh)
    src = attn_arenas(logical, c)
    want = attn_arenas(logical, d)
    dst = filled([a.size for a in want] * replicas)
    oracle.reshard_attn(sh, c, d, src, dst, replicas=replicas)
    for k in range(replicas):
        for t in range(d):
            assert np.array_equal(dst[k * d + t], want[t]), (k, t)
    with pytest.raises(ValueError):
        oracle.reshard_attn(sh, c, d, src, dst[:-1], replicas=replicas)


def test_compact_block_table_in_old_address_order_hand_written():
    """Same two sequences; their old blocks are 7, 2, 5 and 3, 6.  Served in old-id order
    (2, 3, 5, 6, 7) from the free ids 0, 2, 3, 5, 6: old 2 -> 0, 3 -> 2, 5 -> 3, 6 -> 5, 7 -> 6."""
    old = np.array([[7, 2, 5], [3, 6, -1]], np.int32)
    t = oracle.compact_block_table([5, 3], 2, 8, in_use=[1, 4], old_table=old)
    assert t.tolist() == [[6, 0, 3], [2, 5, -1]]
    pairs = sorted((int(old[s, j]), int(t[s, j])) for s in range(2) for j in range(3) if old[s, j] >= 0)
    assert [b for _, b in pairs] == sorted(b for _, b in pairs)          # new ids rise with old ids
