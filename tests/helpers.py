"""Test-side helpers: logical tensors and their sharded arenas written with numpy
indexing (never with byte-offset formulas), used to pin the oracle."""
from __future__ import annotations

import numpy as np

import workloads as W

FILL = 0xCD


def rand_bytes(key, n):
    tags = key if isinstance(key, tuple) else (key,)
    return W.rng.fill_bytes(W.rng.stream_key(0xABCD, *tags), n)


# ---- experts ---------------------------------------------------------------------------

def logical_experts(shape, key=1):
    """uint8 [L, 3, E, m] with independent contents per (l, p, e)."""
    m = shape.d_model * shape.d_ff * shape.elem_bytes
    n = shape.n_layers * 3 * shape.n_experts * m
    return rand_bytes(key, n).reshape(shape.n_layers, 3, shape.n_experts, m)


def expert_arenas(logical, placement, fused_w13=False):
    """Per-rank arena = the rank's experts gathered along the expert axis.  fused_w13:
    per layer a [n][gate|up] tensor (built with numpy.concatenate) and then the [n][down] one."""
    if not fused_w13:
        return [np.ascontiguousarray(logical[:, :, list(p), :]).reshape(-1) for p in placement]
    out = []
    for p in placement:
        mine = logical[:, :, list(p), :]                              # [L, 3, n, m]
        w13 = np.concatenate([mine[:, 0], mine[:, 1]], axis=2)        # [L, n, 2m]
        per_layer = [np.concatenate([w13[l].reshape(-1), mine[l, 2].reshape(-1)])
                     for l in range(mine.shape[0])]
        out.append(np.concatenate(per_layer) if per_layer else np.zeros(0, np.uint8))
    return out


# ---- attention -------------------------------------------------------------------------

def logical_attn(shape, key=2):
    L, D, b = shape.n_layers, shape.d_model, shape.elem_bytes
    q = shape.n_q_heads * shape.head_dim
    kv = shape.n_kv_heads * shape.head_dim
    return dict(
        q=rand_bytes((key, 0), L * q * D * b).reshape(L, q, D * b),
        k=rand_bytes((key, 1), L * kv * D * b).reshape(L, kv, D * b),
        v=rand_bytes((key, 2), L * kv * D * b).reshape(L, kv, D * b),
        o=rand_bytes((key, 3), L * D * q * b).reshape(L, D, q, b),   # [row, column, byte]
    )


def kv_heads_of_rank(n_kv_heads, tp, t):
    """KV heads a TP rank holds: a contiguous share, or - with more ranks than heads -
    the single head floor(t * Hkv / tp) (every head on tp / Hkv consecutive ranks)."""
    n = max(1, n_kv_heads // tp)
    first = t * n_kv_heads // tp
    return list(range(first, first + n))


def _split_kv_rows(x, tp, head_dim):
    """k or v weight [L, Hkv*hd, row bytes] -> per-rank row slices (whole heads)."""
    hkv = x.shape[1] // head_dim
    out = []
    for t in range(tp):
        rows = [h * head_dim + r for h in kv_heads_of_rank(hkv, tp, t) for r in range(head_dim)]
        out.append(x[:, rows])
    return out


def attn_arenas(logical, tp, head_dim=None):
    """Rank t: per layer q_t | k_t | v_t | o_t, pieces cut with numpy.split (k and v by
    whole KV heads when head_dim is given, which also covers tp > Hkv)."""
    L = logical["q"].shape[0]
    qs = np.split(logical["q"], tp, axis=1)
    if head_dim is None:
        ks = np.split(logical["k"], tp, axis=1)
        vs = np.split(logical["v"], tp, axis=1)
    else:
        ks = _split_kv_rows(logical["k"], tp, head_dim)
        vs = _split_kv_rows(logical["v"], tp, head_dim)
    os_ = np.split(logical["o"], tp, axis=2)
    out = []
    for t in range(tp):
        per_layer = [np.concatenate([np.ascontiguousarray(x[l]).reshape(-1)
                                     for x in (qs[t], ks[t], vs[t], os_[t])]) for l in range(L)]
        out.append(np.concatenate(per_layer))
    return out


def attn_arenas_fused_qkv(logical, tp, n_q_heads, n_kv_heads, head_dim):
    """Rank t: per layer [qkv_t | o_t]; qkv_t = for every KV head of the rank, the rank's
    query heads of that head's group, then the k head, then the v head (numpy.concatenate
    of head slices of the logical matrices)."""
    L = logical["q"].shape[0]
    q = logical["q"].reshape(L, n_q_heads, head_dim, -1)
    k = logical["k"].reshape(L, n_kv_heads, head_dim, -1)
    v = logical["v"].reshape(L, n_kv_heads, head_dim, -1)
    os_ = np.split(logical["o"], tp, axis=2)
    q_per_kv = n_q_heads // n_kv_heads
    out = []
    for t in range(tp):
        my_q = list(range(t * n_q_heads // tp, (t + 1) * n_q_heads // tp))
        per_layer = []
        for l in range(L):
            pieces = []
            for g in kv_heads_of_rank(n_kv_heads, tp, t):
                for h in my_q:
                    if h // q_per_kv == g:
                        pieces.append(q[l, h])
                pieces += [k[l, g], v[l, g]]
            per_layer.append(np.concatenate([np.concatenate(pieces).reshape(-1),
                                             np.ascontiguousarray(os_[t][l]).reshape(-1)]))
        out.append(np.concatenate(per_layer))
    return out


# ---- KV --------------------------------------------------------------------------------

def logical_kv(shape, cfg, key=3):
    """uint8 [L, 2, n_logical_blocks, B, Hkv, hd*b]; logical block index runs over
    (sequence, block-in-sequence) in order."""
    B = shape.kv_block_tokens
    nblk = sum(-(-n // B) for n in cfg.seq_lens)
    vec = shape.head_dim * shape.elem_bytes
    n = shape.n_layers * 2 * nblk * B * shape.n_kv_heads * vec
    return rand_bytes(key, n).reshape(shape.n_layers, 2, nblk, B, shape.n_kv_heads, vec)


def kv_arenas(logical, shape, cfg, background=None, head_major=False):
    """Scatters logical blocks into each rank's pool through the block table.  head_major:
    a block is [local head][token][hd] (numpy.swapaxes of the token-major block)."""
    B = shape.kv_block_tokens
    L, vec = shape.n_layers, shape.head_dim * shape.elem_bytes
    hl = max(1, shape.n_kv_heads // cfg.tp)
    phys = []
    for s, n in enumerate(cfg.seq_lens):
        phys += [int(x) for x in cfg.block_table[s, :-(-n // B)]]
    out = []
    for t in range(cfg.tp):
        if background is None:
            pool = np.full((L, 2, cfg.kv_num_blocks, B, hl, vec), FILL, dtype=np.uint8)
        else:
            pool = background[t].reshape(L, 2, cfg.kv_num_blocks, B, hl, vec).copy()
        pool[:, :, phys] = logical[:, :, :, :, kv_heads_of_rank(shape.n_kv_heads, cfg.tp, t)]
        if head_major:
            pool = np.ascontiguousarray(pool.swapaxes(3, 4))
        out.append(pool.reshape(-1))
    return out
