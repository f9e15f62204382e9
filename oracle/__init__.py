"""CPU oracle of the scale-step re-layout (ctypes front of emoe_oracle.cpp).

TEST INFRASTRUCTURE: imported only by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  It never imports the CUDA package, and the CUDA
package never imports it.  Arenas are 1-D numpy uint8 arrays, one per rank.
"""
from __future__ import annotations

import ctypes
from typing import List, Sequence

import numpy as np

from .build import build as _build

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build())
        i32, i64, p = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
        L.emoe_oracle_expert_arena_bytes.restype = i64
        L.emoe_oracle_expert_arena_bytes.argtypes = [i32, i32, i64]
        L.emoe_oracle_attn_arena_bytes.restype = i64
        L.emoe_oracle_attn_arena_bytes.argtypes = [i32] * 7
        L.emoe_oracle_kv_arena_bytes.restype = i64
        L.emoe_oracle_kv_arena_bytes.argtypes = [i32] * 7
        L.emoe_oracle_reshard_experts.restype = i32
        L.emoe_oracle_reshard_experts.argtypes = [i32, i64, i32, p, p, i32, p, p, p, p, i32]
        L.emoe_oracle_reshard_attn.restype = i32
        L.emoe_oracle_reshard_attn.argtypes = [i32] * 8 + [p, p]
        L.emoe_oracle_reshard_kv.restype = i32
        L.emoe_oracle_reshard_kv.argtypes = [i32] * 11 + [p, p, p, p, p, i32]
        L.emoe_oracle_reshard_attn_fused_qkv.restype = i32
        L.emoe_oracle_reshard_attn_fused_qkv.argtypes = [i32] * 8 + [p, p]
        L.emoe_oracle_scaled_expert_scale_base.restype = i64
        L.emoe_oracle_scaled_expert_scale_base.argtypes = [i32, i32, i64]
        L.emoe_oracle_scaled_expert_arena_bytes.restype = i64
        L.emoe_oracle_scaled_expert_arena_bytes.argtypes = [i32, i32, i64, i64]
        L.emoe_oracle_reshard_experts_scaled.restype = i32
        L.emoe_oracle_reshard_experts_scaled.argtypes = [i32, i64, i64, i32, p, p, i32, p, p, p, p]
        L.emoe_oracle_inplace_slots.restype = i32
        L.emoe_oracle_inplace_slots.argtypes = [i32, p, p, i32, p, p, p, p]
        L.emoe_oracle_reshard_experts_inplace.restype = i32
        L.emoe_oracle_reshard_experts_inplace.argtypes = [i32, i64, i32, p, p, i32, p, p, p, p, p]
        _lib = L
    return _lib


def _csr(placement: Sequence[Sequence[int]]):
    off = np.zeros(len(placement) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(p) for p in placement])
    ids = np.array([e for p in placement for e in p], dtype=np.int32)
    return off, ids


def _ptrs(arrs: Sequence[np.ndarray]):
    for a in arrs:
        if a.dtype != np.uint8 or a.ndim != 1 or not a.flags.c_contiguous:
            raise TypeError("arenas must be contiguous 1-D uint8 arrays")
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def _vp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


# ---- arena sizes (bytes) ---------------------------------------------------------------

def expert_arena_bytes(shape, placement) -> List[int]:
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    ms = getattr(shape, "expert_scale_bytes", 0)
    if ms:
        return [lib().emoe_oracle_scaled_expert_arena_bytes(shape.n_layers, len(p), m, ms) for p in placement]
    return [lib().emoe_oracle_expert_arena_bytes(shape.n_layers, len(p), m) for p in placement]


def expert_scale_base(shape, n_slots: int) -> int:
    """Offset of the scale tensor inside the arena of a rank with n_slots experts."""
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    return lib().emoe_oracle_scaled_expert_scale_base(shape.n_layers, n_slots, m)


def attn_arena_bytes(shape, tp: int) -> List[int]:
    n = lib().emoe_oracle_attn_arena_bytes(shape.n_layers, shape.d_model, shape.n_q_heads,
                                          shape.n_kv_heads, shape.head_dim, shape.elem_bytes, tp)
    return [n] * tp


def kv_arena_bytes(shape, tp: int, num_blocks: int) -> List[int]:
    n = lib().emoe_oracle_kv_arena_bytes(shape.n_layers, num_blocks, shape.kv_block_tokens,
                                        shape.n_kv_heads, shape.head_dim, shape.elem_bytes, tp)
    return [n] * tp


# ---- the three phases ------------------------------------------------------------------

def reshard_experts(shape, old_placement, new_placement, src: Sequence[np.ndarray],
                    dst: Sequence[np.ndarray], fused_w13: bool = False) -> None:
    """Writes the new expert arenas `dst` from the old arenas `src` (in place on dst).
    fused_w13: per layer a [n_r][gate|up] tensor followed by a [n_r][down] tensor."""
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    oo, oi = _csr(old_placement)
    no, ni = _csr(new_placement)
    need_s = expert_arena_bytes(shape, old_placement)
    need_d = expert_arena_bytes(shape, new_placement)
    if [a.size for a in src] != need_s or [a.size for a in dst] != need_d:
        raise ValueError("expert arena sizes do not match the placements")
    ms = getattr(shape, "expert_scale_bytes", 0)
    if ms:      # every matrix travels with its scale tensor (weights first, scales after them)
        if fused_w13:
            raise ValueError("oracle: scale tensors go with the plain [L][3][n][m] layout")
        rc = lib().emoe_oracle_reshard_experts_scaled(shape.n_layers, m, ms, len(old_placement), _vp(oo),
                                                     _vp(oi), len(new_placement), _vp(no), _vp(ni),
                                                     _ptrs(src), _ptrs(dst))
        if rc != 0:
            raise ValueError("oracle: an expert of the new placement is absent from the old one")
        return
    rc = lib().emoe_oracle_reshard_experts(shape.n_layers, m, len(old_placement), _vp(oo), _vp(oi),
                                          len(new_placement), _vp(no), _vp(ni), _ptrs(src),
                                          _ptrs(dst), int(bool(fused_w13)))
    if rc != 0:
        raise ValueError("oracle: an expert of the new placement is absent from the old one")


def reshard_attn(shape, tp_old: int, tp_new: int, src, dst, fused_qkv: bool = False,
                 replicas: int = 1) -> None:
    """fused_qkv: per rank and layer one [qkv_t | o_t] arena whose qkv rows are grouped by
    KV head (the group's query heads, then the k head, then the v head).
    replicas > 1: the new side consists of that many data-parallel replicas of the TP group
    (Sec. 5.2 "Attention Weights": added devices receive whole copies of the attention
    tensors); dst lists them replica after replica, tp_new arenas each, and every replica is
    by definition the same re-slice of the old shards."""
    if replicas > 1:
        if len(dst) != tp_new * replicas:
            raise ValueError("attention arena sizes do not match")
        for k in range(replicas):
            reshard_attn(shape, tp_old, tp_new, src, dst[k * tp_new:(k + 1) * tp_new], fused_qkv)
        return
    if ([a.size for a in src] != attn_arena_bytes(shape, tp_old)
            or [a.size for a in dst] != attn_arena_bytes(shape, tp_new)):
        raise ValueError("attention arena sizes do not match")
    fn = lib().emoe_oracle_reshard_attn_fused_qkv if fused_qkv else lib().emoe_oracle_reshard_attn
    rc = fn(shape.n_layers, shape.d_model, shape.n_q_heads,
                                       shape.n_kv_heads, shape.head_dim, shape.elem_bytes,
                                       tp_old, tp_new, _ptrs(src), _ptrs(dst))
    if rc != 0:
        raise ValueError("oracle: TP degree does not divide the head counts")


def reshard_kv(shape, old_cfg, new_cfg, src, dst, head_major: bool = False) -> None:
    """old_cfg / new_cfg carry tp, kv_num_blocks, seq_lens and block_table.
    head_major: blocks are [local head][token][hd] instead of [token][local head][hd]."""
    if ([a.size for a in src] != kv_arena_bytes(shape, old_cfg.tp, old_cfg.kv_num_blocks)
            or [a.size for a in dst] != kv_arena_bytes(shape, new_cfg.tp, new_cfg.kv_num_blocks)):
        raise ValueError("KV arena sizes do not match")
    sl = np.ascontiguousarray(old_cfg.seq_lens, dtype=np.int32)
    if list(sl) != list(new_cfg.seq_lens):
        raise ValueError("old and new configuration list different sequences")
    bo = np.ascontiguousarray(old_cfg.block_table, dtype=np.int32)
    bn = np.ascontiguousarray(new_cfg.block_table, dtype=np.int32)
    if bo.shape != bn.shape:
        w = max(bo.shape[1], bn.shape[1])
        bo = np.pad(bo, ((0, 0), (0, w - bo.shape[1])), constant_values=-1)
        bn = np.pad(bn, ((0, 0), (0, w - bn.shape[1])), constant_values=-1)
    rc = lib().emoe_oracle_reshard_kv(shape.n_layers, shape.kv_block_tokens, shape.n_kv_heads,
                                     shape.head_dim, shape.elem_bytes, old_cfg.tp, new_cfg.tp,
                                     old_cfg.kv_num_blocks, new_cfg.kv_num_blocks, len(sl),
                                     bo.shape[1], _vp(sl), _vp(bo), _vp(bn), _ptrs(src), _ptrs(dst),
                                     int(bool(head_major)))
    if rc != 0:
        raise ValueError("oracle: bad block table or TP degree")


# ---- in-place expert step on capacity-strided arenas ------------------------------------

_INPLACE_ERRORS = {-1: "a wanted expert has no copy in the old slot tables",
                   -2: "a rank has fewer free slots than arrivals",
                   -3: "the capacity of a rank that stays differs between the two sides",
                   -4: "an expert is wanted twice on one rank"}


def inplace_slots(old_slots, want, cap_new) -> List[List[int]]:
    """New slot tables of the in-place expert step.  old_slots: per old rank a list of
    expert ids or -1 (free), its length being the rank's capacity; want: per new rank the
    experts it must hold afterwards; cap_new: capacity per new rank (unchanged for a rank
    that exists on both sides).  Kept experts keep their slot, arrivals take - in the order
    listed - the lowest slot that was free before the step, leaving experts free theirs."""
    oo, oi = _csr(old_slots)
    wo, wi = _csr(want)
    cap = np.ascontiguousarray(cap_new, dtype=np.int32)
    out = np.full(int(cap.sum()), -7, dtype=np.int32)
    rc = lib().emoe_oracle_inplace_slots(len(old_slots), _vp(oo), _vp(oi), len(want), _vp(cap),
                                         _vp(wo), _vp(wi), _vp(out))
    if rc != 0:
        raise ValueError("oracle: " + _INPLACE_ERRORS.get(rc, str(rc)))
    res, b = [], 0
    for c in cap:
        res.append([int(x) for x in out[b:b + c]])
        b += int(c)
    return res


def inplace_arena_bytes(shape, caps) -> List[int]:
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    return [lib().emoe_oracle_expert_arena_bytes(shape.n_layers, int(c), m) for c in caps]


def reshard_experts_inplace(shape, old_slots, want, cap_new, arenas: Sequence[np.ndarray]):
    """Runs the in-place step on `arenas` (max(old ranks, new ranks) arrays, arena r being
    [L][3][cap_r][m]); only arrivals are written.  Returns the new slot tables."""
    new_slots = inplace_slots(old_slots, want, cap_new)
    caps = [len(t) for t in old_slots] + [int(c) for c in list(cap_new)[len(old_slots):]]
    if [a.size for a in arenas] != inplace_arena_bytes(shape, caps):
        raise ValueError("arena sizes do not match the capacities")
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    oo, oi = _csr(old_slots)
    wo, wi = _csr(want)
    cap = np.ascontiguousarray(cap_new, dtype=np.int32)
    flat = np.array([e for t in new_slots for e in t], dtype=np.int32)
    rc = lib().emoe_oracle_reshard_experts_inplace(shape.n_layers, m, len(old_slots), _vp(oo), _vp(oi),
                                                  len(want), _vp(cap), _vp(wo), _vp(wi), _vp(flat),
                                                  _ptrs(arenas))
    if rc != 0:
        raise ValueError("oracle: " + _INPLACE_ERRORS.get(rc, str(rc)))
    return new_slots


# ---- compacting block table ---------------------------------------------------------------

def compact_block_table(seq_lens, block_tokens: int, nb_new: int, in_use=(), old_table=None) -> np.ndarray:
    """The definition of "compacted": going through the sequences in order and through each
    sequence's blocks in order, every block gets the smallest block id of the destination
    pool that is neither in use there already nor handed out before (the paper leaves block
    allocation across instances open, App. C).  Returns int32 [n_seqs, max blocks], -1 padded.
    old_table (same shape of mapped entries): the blocks are served in the order of their OLD
    physical id instead, so that old and new addresses rise together."""
    need = [-(-int(n) // block_tokens) for n in seq_lens]
    out = np.full((len(need), max(need, default=0)), -1, dtype=np.int32)
    taken = set(int(x) for x in in_use)
    todo = [(s, j) for s, n in enumerate(need) for j in range(n)]
    if old_table is not None:
        todo.sort(key=lambda sj: int(old_table[sj[0]][sj[1]]))
    for s, j in todo:
        b = min(x for x in range(nb_new) if x not in taken)    # ValueError if the pool is full
        out[s, j] = b
        taken.add(b)
    return out


# ---- placement chooser: brute force ----------------------------------------------------

def max_kept_bruteforce(n_experts: int, old_placement, ep_new: int) -> int:
    """The most experts any BALANCED placement for ep_new ranks (every expert once, rank
    sizes differing by at most one) leaves on a rank index that already holds a copy
    (Sec. 5.2 "Expert Weights": balance while moving as little as possible).  Exhaustive
    enumeration of all ep_new ** n_experts assignments: tiny inputs only."""
    import itertools
    holds = [set(p) for p in old_placement]
    lo, hi = n_experts // ep_new, -(-n_experts // ep_new)
    best = -1
    for assign in itertools.product(range(ep_new), repeat=n_experts):
        counts = [0] * ep_new
        for r in assign:
            counts[r] += 1
        if min(counts) < lo or max(counts) > hi:
            continue
        kept = sum(1 for e, r in enumerate(assign) if r < len(holds) and e in holds[r])
        best = max(best, kept)
    return best
