// planner.h - host planner of the scale-step re-layout (integer work only).
//
// Turns (model shape, old configuration, new configuration) into per-phase
// copy descriptors.  The plan is a pure function of its inputs, as the paper's
// HMM plan is (Sec. 5.2 "HMM Reconfigures Memory Layout").  No CUDA here.
#pragma once

#include <cstdint>
#include <vector>

#include "../../include/emoe.h"

namespace emoe {

// One destination of a segment.
struct Dst {
  uint64_t off;    // byte offset of run 0 in the destination arena
  uint64_t pitch;  // byte distance between consecutive runs
  uint32_t rank;
  uint32_t pad;
};

// A coalesced, possibly strided, possibly fanned-out copy: n_runs runs of
// run_bytes; run i reads src[src_rank] + src_off + i*src_pitch and is written
// to every destination k at dst[rank_k] + off_k + i*pitch_k.
struct Segment {
  uint64_t src_off;
  uint64_t run_bytes;
  uint64_t src_pitch;
  uint32_t n_runs;
  uint32_t src_rank;
  uint32_t n_dst;
  uint32_t dst_first;  // index of the first destination in PhasePlan::dsts
  uint32_t align;      // largest power of two <= 16 dividing every offset, pitch and run size
  uint32_t pad;
};

struct PhasePlan {
  std::vector<Segment> segs;
  std::vector<Dst> dsts;
  std::vector<uint64_t> arena_old, arena_new;  // bytes per rank
  uint64_t bytes_moved = 0, bytes_read = 0;
  // Every byte the phase writes comes from the same offset of the same rank index, and the
  // arenas have the same sizes: the phase changes nothing (TP kept and, for the KV cache, the
  // block table kept - the paper's zero-copy case).  Set by build_host_plan.
  bool identity = false;
};

// KV phase when the head split changes: block pairs + shape constants.
struct KvPlan {
  std::vector<uint32_t> pair_old, pair_new;  // physical block ids, one entry per mapped block
  uint32_t c = 1, d = 1;                     // old / new TP degree
  uint32_t n_layers = 0, block_tokens = 0, hkv = 0;
  uint64_t head_bytes = 0;                   // head_dim * elem_bytes
  uint64_t nb_old = 0, nb_new = 0;
  bool head_split_changes = false;
  // Heads per rank on either side (1 when a side has more ranks than KV heads) and, for
  // every destination head slot j = new rank * hn + local head, the old rank and local
  // head it is read from.
  uint32_t hc = 0, hn = 0;
  std::vector<uint8_t> src_rank;
  std::vector<uint16_t> src_head;
  bool head_major = false;  // blocks are [local head][token][hd]
  bool replicated = false;  // a side has more ranks than KV heads: the map is not g/hc, g%hc
};

// KV heads of a TP=T group (T <= Hkv: Hkv/T contiguous heads per rank; T > Hkv: one head per
// rank, every head on T/Hkv consecutive ranks) and the old rank a new rank reads head g from.
inline uint32_t kv_heads_per_rank(uint32_t hkv, uint32_t T) { return hkv >= T ? hkv / T : 1u; }
inline uint32_t kv_first_head(uint32_t hkv, uint32_t T, uint32_t t) { return (uint32_t)((uint64_t)t * hkv / T); }
uint32_t kv_source_rank(uint32_t hkv, uint32_t c, uint32_t g, uint32_t r_new);

struct HostPlan {
  emoe_shape_t shape;
  int ep_old, ep_new, tp_old, tp_new;
  uint32_t attn_replicas = 1;  // new attention arenas: tp_new per replica, replica after replica
  uint64_t expert_scale_bytes = 0;  // > 0: expert arenas hold a scale array after a 256-byte-aligned gap
  PhasePlan phase[3];  // experts, attn, kv (kv.segs filled only when the head split is kept)
  KvPlan kv;
};

// Validates and plans.  Returns EMOE_OK or the first validation error.
// flags: the EMOE_LAYOUT_* bits of emoe_plan_create.  expert_scale_bytes: size of the scale
// tensor that goes with every expert matrix (0: none).
// attn_replicas: data-parallel copies of the new TP group that receive the attention shards.
emoe_status_t build_host_plan(const emoe_shape_t &shape, const emoe_config_t &old_cfg,
                              const emoe_config_t &new_cfg, uint32_t flags, uint64_t expert_scale_bytes,
                              uint32_t attn_replicas, HostPlan *out);

// A destination slot that keeps the bytes its rank already holds (paged expert store).
struct Remap {
  uint32_t src_rank, src_slot, dst_rank, dst_slot;
};

// Expert phase for arenas whose slots are `slab` bytes apart (slab >= one matrix).  Slots
// whose source is on the same rank index go to `remaps` instead of being copied.
emoe_status_t build_paged_expert_plan(const emoe_shape_t &shape, const emoe_config_t &old_cfg,
                                      const emoe_config_t &new_cfg, uint64_t slab, PhasePlan *pp,
                                      std::vector<Remap> *remaps);

// In-place expert step on capacity-strided arenas [L][3][cap_r][m] (see
// emoe_plan_create_inplace): segments for arrivals only, and the slot tables after the step.
// arena_old / arena_new of *pp are sized by the capacities; rank r of both sides is the same
// arena when r exists on both.  slab: distance between consecutive slots (0: one matrix; the
// paged store pads every matrix to its allocation granularity).
emoe_status_t build_inplace_expert_plan(const emoe_shape_t &shape, int ep_old, const int32_t *off_old,
                                        const int32_t *ids_old, int ep_new, const int32_t *cap_new,
                                        const int32_t *want_off, const int32_t *want_ids, uint64_t slab,
                                        PhasePlan *pp, std::vector<std::vector<int32_t>> *slot_new);

// Expands a phase into flat emoe_segment_t records (one per destination).  For a
// KV plan with a changing head split the block pairs are expanded per (pair, old
// rank, new rank) overlap.
void export_segments(const HostPlan &hp, int phase, std::vector<emoe_segment_t> *out);

}  // namespace emoe
