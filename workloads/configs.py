"""The five synthetic workloads (C1..C5) and their seeded inputs.

Shapes and reconfigurations follow the benchmark definition of this project
(tiny / mid-size / fine-grained / large-expert-count / overlap).  The
fine-grained and large-expert-count shapes mirror the 64-routed-expert and
128-expert models of the paper's evaluation (Sec. 7.2 "Models and
Baselines"); sequence lengths mirror its request mix of about 2000 prompt
tokens plus 500-750 decode tokens (Sec. 7.6 "SLO Compliance Analysis").  Trained weights and request
traces are not needed: the path moves bytes and never looks at them.

Nothing in this module computes a re-layout: placements and block tables are
*inputs* of the method, and arena contents are filled by physical position.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from . import rng

MASTER_SEED = 0xE1A571C0

# stream tags
TAG_VALUES, TAG_BT_OLD, TAG_BT_NEW, TAG_SEQLEN, TAG_ZIPF_DRAW, TAG_ZIPF_PERM = range(6)
# arena kinds (second tag of a value stream)
KIND_EXPERTS, KIND_ATTN, KIND_KV = range(3)


@dataclass(frozen=True)
class Shape:
    n_layers: int
    n_routed: int
    n_shared: int
    d_model: int
    d_ff: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    kv_block_tokens: int = 16
    elem_bytes: int = 2
    expert_scale_bytes: int = 0   # bytes of the scale tensor that goes with every expert matrix (0: none)

    @property
    def n_experts(self) -> int:
        return self.n_routed + self.n_shared


@dataclass
class ParallelConfig:
    ep: int
    tp: int
    placement: List[List[int]]            # expert ids per EP rank, slot order
    kv_num_blocks: int                    # pool size per (layer, K|V) per TP rank
    seq_lens: List[int]
    block_table: np.ndarray               # int32 [n_seqs, max_blocks], -1 padded


@dataclass
class Workload:
    name: str
    shape: Shape
    old: ParallelConfig
    new: ParallelConfig
    seed: int
    notes: str = ""
    victim: Optional[dict] = field(default=None)   # C5: the concurrent GEMM's shape
    fused_w13: bool = False        # layout variant: per layer [n][gate|up] then [n][down]
    kv_head_major: bool = False    # layout variant: KV blocks [local head][token][hd]
    fused_qkv: bool = False        # layout variant: attention arena [qkv_t | o_t], rows grouped by KV head
    attn_replicas: int = 1         # data-parallel replicas of the new TP group that receive the attention shards

    def with_layers(self, n_layers: int) -> "Workload":
        """Same workload cut to n_layers (layers are independent in every phase)."""
        return dataclasses.replace(self, shape=dataclasses.replace(self.shape, n_layers=n_layers))

    def swapped(self) -> "Workload":
        """The inverse reconfiguration (new -> old), for round trips."""
        return dataclasses.replace(self, old=self.new, new=self.old, name=self.name + "_inverse")


# ---- placement generators (inputs of the method) ---------------------------------------

def place_round_robin(n_experts: int, ep: int) -> List[List[int]]:
    """Expert e on rank e mod ep, slot e div ep."""
    return [list(range(r, n_experts, ep)) for r in range(ep)]


def place_contiguous(n_experts: int, ep: int) -> List[List[int]]:
    """Balanced id ranges: the first n_experts mod ep ranks hold one expert more."""
    base, extra = divmod(n_experts, ep)
    out, e = [], 0
    for r in range(ep):
        n = base + (1 if r < extra else 0)
        out.append(list(range(e, e + n)))
        e += n
    return out


def with_shared(placement: List[List[int]], shared_ids: List[int]) -> List[List[int]]:
    """Shared experts appended after the routed slots of every rank."""
    return [list(p) + list(shared_ids) for p in placement]


def zipf_load(seed: int, n_experts: int, alpha: float = 1.2, draws: int = 1 << 20) -> np.ndarray:
    """Router load per expert: `draws` samples of p(k) ~ k^-alpha over popularity
    ranks k = 1..n_experts (inverse CDF on the counter stream); popularity rank
    -> expert id by a seeded permutation."""
    p = np.arange(1, n_experts + 1, dtype=np.float64) ** -alpha
    cdf = np.cumsum(p / p.sum())
    cdf[-1] = 1.0
    u = rng.uniform01(rng.stream_key(seed, TAG_ZIPF_DRAW), 0, draws)
    ranks = np.searchsorted(cdf, u, side="right")
    counts_by_rank = np.bincount(ranks, minlength=n_experts)[:n_experts]
    perm = rng.permutation(rng.stream_key(seed, TAG_ZIPF_PERM), n_experts)
    load = np.zeros(n_experts, dtype=np.int64)
    load[perm] = counts_by_rank
    return load


def place_hot_replicated(load: np.ndarray, ep: int, n_hot: int) -> List[List[int]]:
    """The n_hot most loaded experts get two instances (each at half load); all
    instances are assigned longest-processing-time-first to the least loaded
    rank that has capacity and does not hold that expert yet; slots by id."""
    n = len(load)
    order = sorted(range(n), key=lambda e: (-int(load[e]), e))
    hot = set(order[:n_hot])
    inst = []
    for e in range(n):
        if e in hot:
            inst += [(load[e] / 2.0, e), (load[e] / 2.0, e)]
        else:
            inst.append((float(load[e]), e))
    inst.sort(key=lambda t: (-t[0], t[1]))
    cap = -(-len(inst) // ep)
    ranks: List[List[int]] = [[] for _ in range(ep)]
    tot = [0.0] * ep
    for w, e in inst:
        cands = [r for r in range(ep) if len(ranks[r]) < cap and e not in ranks[r]]
        r = min(cands, key=lambda r: (tot[r], r))
        ranks[r].append(e)
        tot[r] += w
    return [sorted(p) for p in ranks]


# ---- block tables ----------------------------------------------------------------------

def make_seq_lens(seed: int, total_blocks: int, block_tokens: int,
                  lo: int = 2000, hi: int = 2750) -> List[int]:
    """Sequence lengths uniform in [lo, hi] appended until the block budget is
    used up; the last sequence is truncated to the blocks that remain."""
    key = rng.stream_key(seed, TAG_SEQLEN)
    out, left, i = [], total_blocks, 0
    while left > 0:
        n = lo + int(rng.hash_u64(key, i, 1)[0] % np.uint64(hi - lo + 1))
        n = min(n, left * block_tokens)
        out.append(n)
        left -= -(-n // block_tokens)
        i += 1
    return out


def make_block_table(key: int, seq_lens: List[int], block_tokens: int, pool: int,
                     order: str = "random") -> np.ndarray:
    """Assigns distinct physical blocks of a pool to the sequences' logical
    blocks: a seeded random permutation of the pool, or identity (compacting)."""
    nblk = [-(-n // block_tokens) for n in seq_lens]
    used = sum(nblk)
    if used > pool:
        raise ValueError("pool smaller than the blocks in use")
    ids = rng.permutation(key, pool)[:used] if order == "random" else np.arange(used)
    bt = np.full((len(seq_lens), max(nblk)), -1, dtype=np.int32)
    p = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = ids[p:p + n]
        p += n
    return bt


def _kv_configs(seed: int, total_blocks: int, block_tokens: int, seq_lens: Optional[List[int]],
                slack: float = 0.125, new_order: str = "random"):
    if seq_lens is None:
        seq_lens = make_seq_lens(seed, total_blocks, block_tokens)
    nb_old = total_blocks
    nb_new = total_blocks + int(total_blocks * slack)
    bt_old = make_block_table(rng.stream_key(seed, TAG_BT_OLD), seq_lens, block_tokens, nb_old)
    bt_new = make_block_table(rng.stream_key(seed, TAG_BT_NEW), seq_lens, block_tokens, nb_new,
                              order=new_order)
    return seq_lens, nb_old, bt_old, nb_new, bt_new


# ---- the five workloads ----------------------------------------------------------------

WORKLOAD_NAMES = ("c1_tiny", "c2_mid", "c3_fine", "c4_large", "c5_overlap")
# beyond the five benchmark configurations: shaped like the largest model of the paper's
# evaluation (256 routed experts, wider d_model, FP8 weights with block scales), cut to the
# layers that fit one GPU
EXTRA_WORKLOAD_NAMES = ("c6_wide_fp8",)


def make_workload(name: str, n_layers: Optional[int] = None, new_order: str = "random") -> Workload:
    if name == "c1_tiny":
        seed = MASTER_SEED + 0
        sh = Shape(4, 8, 0, 256, 512, 8, 8, 32)
        sl, nbo, bto, nbn, btn = _kv_configs(seed, 64, 16, [256] * 4, new_order=new_order)
        old = ParallelConfig(2, 1, place_round_robin(8, 2), nbo, sl, bto)
        new = ParallelConfig(4, 2, place_round_robin(8, 4), nbn, sl, btn)
        notes = "EP2,TP1 -> EP4,TP2, round-robin placement"
    elif name == "c2_mid":
        seed = MASTER_SEED + 1
        sh = Shape(24, 60, 0, 2048, 1408, 16, 16, 128)
        sl, nbo, bto, nbn, btn = _kv_configs(seed, 32768 // 16, 16, None, new_order=new_order)
        old = ParallelConfig(4, 1, place_contiguous(60, 4), nbo, sl, bto)
        new = ParallelConfig(6, 1, place_contiguous(60, 6), nbn, sl, btn)
        notes = "EP4 -> EP6, contiguous expert ranges, TP1"
    elif name in ("c3_fine", "c5_overlap"):
        seed = MASTER_SEED + 2
        sh = Shape(27, 64, 2, 2048, 1408, 16, 16, 128)
        sl, nbo, bto, nbn, btn = _kv_configs(seed, 65536 // 16, 16, None, new_order=new_order)
        old = ParallelConfig(8, 1, with_shared(place_contiguous(64, 8), [64, 65]), nbo, sl, bto)
        new = ParallelConfig(12, 1, with_shared(place_contiguous(64, 12), [64, 65]), nbn, sl, btn)
        notes = "EP8 -> EP12 uneven (6,6,6,6,5,..), 2 shared experts on every rank, TP1"
    elif name == "c4_large":
        seed = MASTER_SEED + 3
        sh = Shape(16, 128, 0, 2048, 768, 32, 4, 128)
        sl, nbo, bto, nbn, btn = _kv_configs(seed, 131072 // 16, 16, None, new_order=new_order)
        load = zipf_load(seed, 128, 1.2)
        old = ParallelConfig(3, 2, place_contiguous(128, 3), nbo, sl, bto)
        new = ParallelConfig(5, 4, place_hot_replicated(load, 5, 8), nbn, sl, btn)
        notes = "EP3 -> EP5 with the 8 hottest experts (Zipf 1.2) held twice; TP2 -> TP4"
    elif name == "c6_wide_fp8":
        # 256 routed experts + 1 shared, d_model 7168, expert d_ff 2048, one byte per weight and
        # one fp32 scale per 128 x 128 block (56 x 16 x 4 bytes per matrix); 5 of the model's
        # layers: old + new expert arenas are then 117 GB
        seed = MASTER_SEED + 5
        sh = Shape(5, 256, 1, 7168, 2048, 128, 8, 128, 16, 1, 56 * 16 * 4)
        sl, nbo, bto, nbn, btn = _kv_configs(seed, 65536 // 16, 16, None, new_order=new_order)
        old = ParallelConfig(8, 1, with_shared(place_contiguous(256, 8), [256]), nbo, sl, bto)
        new = ParallelConfig(12, 1, with_shared(place_contiguous(256, 12), [256]), nbn, sl, btn)
        notes = ("EP8 -> EP12, 256 routed experts + 1 shared on every rank, FP8 weights with "
                 "128x128-block fp32 scales moved by the same plan, TP1")
    else:
        raise KeyError(name)
    victim = None
    if name == "c5_overlap":
        victim = dict(active_experts=8, tokens=256, top_k=8, d_model=2048, d_ff=1408)
        notes += "; reshard on a low-priority stream beside a grouped expert GEMM"
    wl = Workload(name, sh, old, new, seed, notes, victim)
    if n_layers is not None:
        wl = wl.with_layers(n_layers)
    return wl


def make_exchange_workload(n_devices: int, n_layers: Optional[int] = None) -> Workload:
    """A scale step whose ranks map onto n_devices GPUs, one rank index per GPU: the
    fine-grained shape (64 routed + 2 shared experts), expert parallelism grown by two devices
    as in the paper's step pattern (n_devices - 2 -> n_devices; 1 -> 2 for two devices),
    tensor parallelism doubled (n_devices / 2 -> n_devices, capped by the 16 heads), so
    experts, attention slices and KV heads all cross devices."""
    if n_devices < 2 or n_devices > 16 or n_devices & (n_devices - 1):
        raise ValueError("exchange workloads are defined for 2, 4, 8 or 16 devices")
    seed = MASTER_SEED + 6
    sh = Shape(27, 64, 2, 2048, 1408, 16, 16, 128)
    sl, nbo, bto, nbn, btn = _kv_configs(seed, 65536 // 16, 16, None)
    ep_old = n_devices - 2 if n_devices >= 4 else 1
    old = ParallelConfig(ep_old, n_devices // 2, with_shared(place_contiguous(64, ep_old), [64, 65]), nbo, sl, bto)
    new = ParallelConfig(n_devices, n_devices, with_shared(place_contiguous(64, n_devices), [64, 65]), nbn, sl, btn)
    wl = Workload("exchange_%d" % n_devices, sh, old, new, seed,
                  "EP%d,TP%d -> EP%d,TP%d, one rank per GPU, pulled over the GPU interconnect"
                  % (ep_old, n_devices // 2, n_devices, n_devices))
    return wl.with_layers(n_layers) if n_layers is not None else wl


def small_variant(name: str) -> Workload:
    """A few-layer cut of a workload with the same per-layer structure, sized so
    that a CPU implementation finishes in seconds."""
    return make_workload(name, n_layers={"c1_tiny": 4}.get(name, 1))


def arena_key(wl_seed: int, kind: int, rank: int) -> int:
    """Key of the value stream that fills one old-layout arena by byte position."""
    return rng.stream_key(wl_seed, TAG_VALUES, kind, rank)
