// kernels.h - launch interface of the sm_100a copy kernels.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

#include "planner.h"

namespace emoe {

// A schedulable piece of one segment: n_tiles consecutive tiles starting at
// first_tile.  A tile is either a chunk of at most tile_bytes of one long run,
// or as many whole short runs ("rows") as fit into tile_bytes.
struct Unit {
  uint32_t seg;
  uint32_t first_tile;
  uint32_t n_tiles;
  uint32_t pad;
};

constexpr int kMaxFanout = 8;  // destinations one bulk tile is stored to (longer lists are split)

struct RankPtrs {
  const uint8_t *src[EMOE_MAX_RANKS];
  uint8_t *dst[EMOE_MAX_RANKS];
};

// Device-side copy descriptor: a planner Segment with its first destination inlined, so
// that the common one-destination case needs no second table look-up.  With n_dst > 1
// all destinations (the first included) are dsts[dst_first .. dst_first + n_dst).
struct DevSeg {
  uint64_t src_off, run_bytes, src_pitch;
  uint64_t dst_off, dst_pitch;
  uint32_t n_runs, src_rank, dst_rank, n_dst, dst_first, align;
};
static_assert(sizeof(DevSeg) == 64, "DevSeg is read as four 16-byte words");

struct SegTables {  // device pointers
  const DevSeg *segs;
  const Dst *dsts;
  const Unit *units;
  uint32_t n_units;
};

constexpr uint32_t kKvMapMax = 64;  // destination head slots a replicated split can have

struct KvTables {  // device pointers + shape constants of the KV head re-split
  const uint32_t *pair_old, *pair_new;
  uint32_t n_pairs, n_lk;        // n_lk = 2 * n_layers
  uint32_t block_tokens;
  uint32_t hkv;                  // destination head slots per token: new ranks x heads per new rank
                                 // (= the KV head count unless the new side replicates heads)
  uint32_t hc, hn;               // heads per old / new rank
  uint32_t head_bytes;
  uint64_t nb_old, nb_new;
  // With more ranks than KV heads on a side, slot j = new rank * hn + local head reads
  // old rank map_rank[j], local head map_head[j]; otherwise slot j is global head j and
  // lives at old rank j / hc, local head j % hc.
  uint32_t use_map;
  uint32_t dst_only;             // write only this new rank's blocks (0xffffffff: all ranks)
  uint8_t map_rank[kKvMapMax], map_head[kKvMapMax];
};

struct BulkConfig {
  uint32_t tile_bytes, stages, hints;
  uint32_t pace_ns;             // least time between a CTA's full-tile loads; 0 = unpaced
  unsigned long long wait_ns;   // bound of every device-side wait
};
// Dynamic shared memory the bulk kernel needs / may use at most.
size_t bulk_smem_bytes(uint32_t tile_bytes, uint32_t stages);
size_t bulk_smem_limit();
// Bulk path: cp.async.bulk global -> shared -> global through an mbarrier ring.
// ctr: two zero-initialised words in device memory through which the CTAs of ONE launch
// claim units (they leave them at zero); launches that may run at the same time need
// different words.  null: units are dealt round-robin.
cudaError_t launch_bulk_copy(const SegTables &t, const RankPtrs &ptrs, const BulkConfig &c,
                             uint32_t grid, int *status, unsigned int *ctr, cudaStream_t stream);
// Vector path: a warp per tile, 16-byte (or narrower, per segment alignment) loads and stores.
cudaError_t launch_vec_copy(const SegTables &t, const RankPtrs &ptrs, uint32_t tile_bytes,
                            uint32_t grid, cudaStream_t stream);
// KV head re-split; mode 1 = direct register copy, mode 2 = staged through shared memory,
// mode 3 = tiled TMA loads and stores (each falls back to direct where it does not apply).
// grid = CTA budget in SMs; unbounded = no budget was set (the direct kernels then launch
// one CTA per tile).
constexpr uint32_t kKvTmaMaxRanks = 12;  // tensor maps travel in the kernel parameters
bool kv_staged_supported(const KvTables &t, uint32_t *stages_out);
bool kv_tma_supported(const KvTables &t, uint32_t *stages_out);
cudaError_t launch_kv_copy(const KvTables &t, const RankPtrs &ptrs, int mode, uint32_t grid,
                           bool unbounded, int *status, unsigned long long wait_ns,
                           cudaStream_t stream);
// The vector path and the direct KV head re-split in ONE launch (head vectors must be
// multiples of 16 bytes: vec_kv_supported).  grid / unbounded as for launch_kv_copy.
bool vec_kv_supported(const KvTables &kv);
cudaError_t launch_vec_kv_copy(const SegTables &t, const RankPtrs &ptrs, uint32_t tile_bytes,
                               const KvTables &kv, const RankPtrs &kv_ptrs, uint32_t grid,
                               bool unbounded, cudaStream_t stream);

// KV head re-split with its block-pair list in a fixed __device__ array of the library
// image (no allocation).  pair_old / pair_new: host arrays of n_pairs ids.  Returns
// EMOE_OK, EMOE_ERR_TOO_LARGE (n_pairs > EMOE_STATIC_KV_MAX_PAIRS) or EMOE_ERR_CUDA.
emoe_status_t launch_kv_copy_static(const KvTables &shape_only, const uint32_t *pair_old,
                                    const uint32_t *pair_new, const RankPtrs &ptrs,
                                    cudaStream_t stream);

// Writes the regular unit table of a phase on the device.  Runs are taken `group` at a time
// (group > 1 only for runs of fewer tiles than a unit: those runs then form ONE unit); for
// every group g and every listed segment k (index seg_idx[k] + seg_offset into segs) the
// units of that group go to out[g * units_per_group + seg_pre[k] ...], each of at most
// unit_tiles tiles of tile_bytes.
cudaError_t launch_gen_units(const DevSeg *segs, const uint32_t *seg_idx, const uint32_t *seg_pre,
                             uint32_t n_segs, uint32_t n_runs, uint32_t group, uint32_t units_per_group,
                             uint32_t tile_bytes, uint32_t unit_tiles, uint32_t seg_offset, Unit *out,
                             cudaStream_t stream);

// Kernel attribute setup (dynamic shared memory opt-in) for the CURRENT device; cheap after
// the first call on a device.
cudaError_t kernels_init();

}  // namespace emoe
