// capi.cpp - the C ABI of libemoe.so: plan life cycle, argument checks, launches.
#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "internal.h"
#include "kernels.h"
#include "planner.h"

using namespace emoe;

namespace {

// A named range around an entry point, for timelines of profilers that follow NVTX (a no-op
// costing a few nanoseconds when no such tool is attached).
struct TraceRange {
  explicit TraceRange(const char *name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange &) = delete;
  TraceRange &operator=(const TraceRange &) = delete;
};

constexpr uint32_t kUnitTiles = 8;
constexpr uint32_t kDefaultBulkTile = 32768, kDefaultBulkStages = 6;
constexpr uint32_t kDefaultHints = 0;
constexpr int kCtrSlots = 4;        // launches of one phase of one plan that may be in flight at once
constexpr int kTableSets = 4;        // experts, attn, kv, and the three merged for one whole step
constexpr int kStatusWords = 1 + kTableSets * kCtrSlots * 2;
constexpr int kDefaultKvMode = 1;   // 1 direct, 2 staged through shared memory
constexpr int kDefaultKvOrder = 2;  // 1 table order, 2 by old block id (sequential reads: measured best), 3 by new block id
constexpr uint32_t kDefaultBulkCtas = 74;  // measured optimum on B200: half the SMs, deep rings
constexpr uint32_t kVecTile = 16384;
constexpr uint64_t kBulkMinRun = 16384;  // shorter runs go to the vector kernel
constexpr unsigned long long kDefaultWaitNs = 4000000000ull;  // bound of a device-side wait: 4 s
constexpr uint64_t kMergeBulkBelow = 1ull << 30;   // see build_tables
constexpr uint64_t kSmallPhaseBytes = 256ull << 20;

struct DevPhase {
  std::vector<DevSeg> segs;  // routed copy of the host segments (fan-out split to kMaxFanout)
  std::vector<Dst> dsts;
  std::vector<Unit> bulk_units, vec_units;   // bulk_units: the host-built part only (see n_gen)
  uint64_t n_bulk = 0;                        // bulk units of the phase: n_gen + bulk_units.size()
  // The first n_gen bulk units - those of the "regular" segments: the same number of runs
  // each, every run at least a tile long - are expanded on the device from these (segment
  // indices, offset of each one's units inside a run, runs per segment, units per run); the
  // units of the other bulk segments are built on the host and follow them.
  uint64_t n_gen = 0;
  std::vector<uint32_t> gen_seg, gen_pre;
  uint32_t gen_runs = 0, gen_upr = 0, gen_group = 1;   // gen_upr: units per group of gen_group runs
  uint64_t rest_off[3] = {0, 0, 0};           // merged set: where each phase's host-built units start in bulk_units
  DevSeg *d_segs = nullptr;
  Dst *d_dsts = nullptr;
  Unit *d_bulk_units = nullptr, *d_vec_units = nullptr;
};

}  // namespace

// State of the pipelined host-buffer step (EMOE_PLAN_HOST_STEP): plans for a chunk of
// layers (layers are independent in every phase and every arena is layer-major, so a
// plan for lc layers applied to pointers advanced by whole layers does exactly those
// layers), two copy streams and the events that order copy-in -> kernels -> copy-out.
struct HostStep {
  emoe_plan *chunk = nullptr, *tail = nullptr;  // plans for lc layers / for the last L % lc layers
  int lc = 0, n_chunks = 0;                     // n_chunks counts the tail chunk too
  cudaStream_t s_in = nullptr, s_out = nullptr;
  std::vector<cudaEvent_t> ev_in, ev_k;
  cudaEvent_t ev_start = nullptr, ev_done = nullptr;
};

struct emoe_plan {
  HostPlan hp;
  HostStep *hs = nullptr;
  bool host_only = true;
  int device = -1, sm_count = 148;
  emoe_tuning_t tuning{};
  bool inplace = false;           // expert step on capacity-strided arenas (emoe_plan_create_inplace)
  std::vector<std::vector<int32_t>> slot_new;   // ... its slot tables after the step
  int local_rank = -1;            // >= 0: only destinations of this new-rank index are written
  bool reads_src[3][EMOE_MAX_RANKS];  // old ranks the (filtered) phase reads
  DevPhase dev[kTableSets];       // [3]: all three phases as one launch set (see build_merged)
  uint32_t src_base[3] = {0, 0, 0}, dst_base[3] = {0, 0, 0};  // rank offsets of a phase in the merged set
  bool merged = false;
  uint32_t merged_seg0[3] = {0, 0, 0};        // first segment / first bulk unit of a phase in the merged set
  uint64_t merged_unit0[3] = {0, 0, 0};
  std::vector<uint32_t> pair_old, pair_new;  // block pairs in launch order (see kv_order)
  uint32_t *d_pair_old = nullptr, *d_pair_new = nullptr;
  int *d_status = nullptr;  // [0] status word; then kCtrSlots x 2 work-counter words per phase
  mutable std::atomic<uint32_t> launch_seq[kTableSets];
  // A whole step with two launch sets runs them side by side: the second set goes to a
  // stream of the plan's own, forked from and joined to the caller's stream with events.
  // side[0] has the least priority, side[1] the greatest; the one nearer the caller's
  // stream is used.  The mutex orders the record / wait pairs of concurrent callers.
  cudaStream_t side[2] = {nullptr, nullptr};
  int prio_least = 0, prio_greatest = 0;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  mutable std::mutex fork_mu;
  emoe_plan() { for (auto &a : launch_seq) a.store(0); }
};

namespace {

uint32_t bulk_tile(const emoe_plan *p) {
  return p->tuning.bulk_tile_bytes > 0 ? (uint32_t)p->tuning.bulk_tile_bytes : kDefaultBulkTile;
}
uint32_t bulk_stages(const emoe_plan *p) {
  return p->tuning.bulk_stages > 0 ? (uint32_t)p->tuning.bulk_stages : kDefaultBulkStages;
}
uint64_t bulk_min_run(const emoe_plan *p) {
  return p->tuning.bulk_min_run > 0 ? (uint64_t)p->tuning.bulk_min_run : kBulkMinRun;
}
// Bound of the device-side waits in ns; 0 = a wait that is not satisfied at once fails.
unsigned long long wait_ns(const emoe_plan *p) {
  if (p->tuning.wait_limit_us < 0) return 0;
  return p->tuning.wait_limit_us > 0 ? (unsigned long long)p->tuning.wait_limit_us * 1000ull : kDefaultWaitNs;
}
int kv_mode(const emoe_plan *p) { return p->tuning.kv_mode > 0 ? p->tuning.kv_mode : kDefaultKvMode; }
// The KV head re-split shares a launch with the vector work when it uses the direct copy.
bool fused_kv(const emoe_plan *p, const KvTables &t) {
  return (kv_mode(p) == 1 || kv_mode(p) == 4) && p->tuning.serial < 2 && vec_kv_supported(t);
}
int kv_order(const emoe_plan *p) {
  return p->tuning.kv_order > 0 ? p->tuning.kv_order : kDefaultKvOrder;
}

// Cuts one segment into units of at most kUnitTiles tiles and hands each to f(first run
// the unit touches, unit).  A unit of a long-run segment (run >= tile) whose runs fill a unit
// stays inside one run, so that units can be ordered by run; runs of fewer tiles than a unit
// (a 64 KiB KV block is two) are taken several to a unit - runs_per_unit() consecutive runs -
// because a unit is the grain at which CTAs claim work and fetch descriptors, and a grain of
// two tiles costs 4-5 % of the bandwidth.
uint32_t runs_per_unit(uint32_t tiles_per_run) {
  return tiles_per_run >= kUnitTiles ? 1u : kUnitTiles / tiles_per_run;
}

template <typename F>
void for_each_unit(uint32_t seg, const DevSeg &s, uint32_t T, F &&f) {
  if (s.run_bytes >= T) {
    const uint32_t tpr = (uint32_t)((s.run_bytes + T - 1) / T);
    const uint32_t g = runs_per_unit(tpr);
    if (g > 1) {
      for (uint32_t run = 0; run < s.n_runs; run += g) {
        const uint32_t n = s.n_runs - run < g ? s.n_runs - run : g;
        f(run, Unit{seg, run * tpr, n * tpr, 0});
      }
      return;
    }
    for (uint32_t run = 0; run < s.n_runs; ++run)
      for (uint32_t t = 0; t < tpr; t += kUnitTiles) {
        const uint32_t n = tpr - t < kUnitTiles ? tpr - t : kUnitTiles;
        f(run, Unit{seg, run * tpr + t, n, 0});
      }
  } else {
    const uint32_t rpt = (uint32_t)(T / s.run_bytes);
    const uint32_t n_tiles = (s.n_runs + rpt - 1) / rpt;
    for (uint32_t t = 0; t < n_tiles; t += kUnitTiles) {
      const uint32_t n = n_tiles - t < kUnitTiles ? n_tiles - t : kUnitTiles;
      f(t * rpt, Unit{seg, t, n, 0});
    }
  }
}

// The general case: the bulk unit table written on the host, run-major without a sort
// (count the units of every run, turn the counts into start positions, then place).
void expand_units_on_host(DevPhase *dp, const std::vector<uint32_t> &bulk_segs, uint32_t T, bool run_major) {
  dp->bulk_units.clear();
  if (run_major) {
    uint32_t max_run = 0;
    for (uint32_t idx : bulk_segs) max_run = std::max(max_run, dp->segs[idx].n_runs);
    std::vector<uint32_t> start((size_t)max_run + 2, 0);
    for (uint32_t idx : bulk_segs)
      for_each_unit(idx, dp->segs[idx], T, [&](uint32_t run, const Unit &) { start[run + 1]++; });
    for (size_t i = 1; i < start.size(); ++i) start[i] += start[i - 1];
    dp->bulk_units.resize(start.back());
    for (uint32_t idx : bulk_segs)
      for_each_unit(idx, dp->segs[idx], T, [&](uint32_t run, const Unit &u) { dp->bulk_units[start[run]++] = u; });
  } else {
    for (uint32_t idx : bulk_segs)
      for_each_unit(idx, dp->segs[idx], T, [&](uint32_t, const Unit &u) { dp->bulk_units.push_back(u); });
  }
}

// Routes every host segment to the bulk or the vector kernel and cuts it into units.
//
// Launch order of the bulk units is run-major: all segments' run 0, then all segments'
// run 1, ...  Runs of one segment are a pitch apart (a whole layer slab, a whole KV pool),
// so this keeps the CTAs that run at the same time inside one slab - sequential DRAM
// pages and a small TLB footprint - instead of spread over the whole arena.
void build_tables(emoe_plan *p, int phase) {
  const PhasePlan &pp = p->hp.phase[phase];
  DevPhase &dp = p->dev[phase];
  dp.segs.clear(); dp.dsts.clear(); dp.bulk_units.clear(); dp.vec_units.clear();
  dp.gen_seg.clear(); dp.gen_pre.clear();
  dp.n_gen = 0; dp.n_bulk = 0; dp.gen_runs = dp.gen_upr = 0; dp.gen_group = 1;
  for (bool &b : p->reads_src[phase]) b = false;
  const uint32_t T = bulk_tile(p);

  // KV with the head split kept: one segment per block pair and TP rank.  Visit them in
  // the order kv_order asks for (old or new physical block order instead of table order).
  std::vector<uint32_t> order(pp.segs.size());
  for (uint32_t i = 0; i < order.size(); ++i) order[i] = i;
  if (phase == EMOE_PHASE_KV && kv_order(p) >= 2) {
    const bool by_new = kv_order(p) == 3;
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
      const Segment &x = pp.segs[a], &y = pp.segs[b];
      const uint64_t kx = by_new ? pp.dsts[x.dst_first].off : x.src_off;
      const uint64_t ky = by_new ? pp.dsts[y.dst_first].off : y.src_off;
      return kx != ky ? kx < ky : x.src_rank < y.src_rank;
    });
  }

  // Default routing: long aligned runs to the bulk kernel, the rest to the vector kernel.
  // A phase that is small, or that needs the vector kernel anyway and has little bulk
  // work, goes to the vector kernel whole: one launch instead of two, and a short bulk
  // launch never gets past its ramp-up (measured on the attention phase: 5.3 -> 5.9 TB/s).
  uint64_t bulk_bytes = 0, vec_bytes = 0;
  for (const Segment &s0 : pp.segs) {
    const uint64_t b = (uint64_t)s0.n_runs * s0.run_bytes * s0.n_dst;
    if (s0.align == 16 && s0.run_bytes >= bulk_min_run(p)) bulk_bytes += b; else vec_bytes += b;
  }
  const bool all_vec = p->tuning.path == 0 &&
                       ((vec_bytes > 0 && bulk_bytes < kMergeBulkBelow) ||
                        bulk_bytes + vec_bytes < kSmallPhaseBytes);

  std::vector<uint32_t> bulk_segs;  // indices into dp.segs of the segments the bulk kernel takes
  Dst mine[EMOE_MAX_RANKS];
  for (uint32_t oi : order) {
    const Segment &s0 = pp.segs[oi];
    bool is_bulk = s0.align == 16 && s0.run_bytes >= bulk_min_run(p) && !all_vec;
    if (p->tuning.path == 1) is_bulk = false;
    if (p->tuning.path == 2) is_bulk = (s0.align == 16);
    // destinations this plan writes: all, or those of the local rank only (a source has at
    // most one destination per rank, so EMOE_MAX_RANKS entries suffice)
    uint32_t n_mine = 0;
    for (uint32_t j = 0; j < s0.n_dst; ++j) {
      const Dst &d = pp.dsts[s0.dst_first + j];
      if ((p->local_rank < 0 || (int)d.rank == p->local_rank) && n_mine < EMOE_MAX_RANKS) mine[n_mine++] = d;
    }
    if (n_mine == 0) continue;
    p->reads_src[phase][s0.src_rank] = true;
    const uint32_t max_fan = is_bulk ? (uint32_t)kMaxFanout : n_mine;
    for (uint32_t k = 0; k < n_mine; k += max_fan) {
      DevSeg s{};
      s.src_off = s0.src_off; s.run_bytes = s0.run_bytes; s.src_pitch = s0.src_pitch;
      s.n_runs = s0.n_runs; s.src_rank = s0.src_rank; s.align = s0.align;
      s.n_dst = n_mine - k < max_fan ? n_mine - k : max_fan;
      s.dst_first = (uint32_t)dp.dsts.size();
      const Dst &d0 = mine[k];
      s.dst_off = d0.off; s.dst_pitch = d0.pitch; s.dst_rank = d0.rank;
      if (s.n_dst > 1)  // the one-destination case reads the inlined copy only
        for (uint32_t j = 0; j < s.n_dst; ++j) dp.dsts.push_back(mine[k + j]);
      const uint32_t idx = (uint32_t)dp.segs.size();
      dp.segs.push_back(s);
      if (is_bulk) bulk_segs.push_back(idx);
      else for_each_unit(idx, s, kVecTile, [&](uint32_t, const Unit &u) { dp.vec_units.push_back(u); });
    }
  }
  // Bulk units in run-major order.  The regular segments (run >= tile, and as many runs as the
  // first such segment - all long runs of the bench phases) only get their offset inside a run
  // computed here: that part of the table is written by a kernel at upload time.  The units of
  // the remaining bulk segments (short rows packed into tiles, other run counts) are few and
  // are built here; they follow the generated part.
  std::vector<uint32_t> rest;
  if (p->tuning.unit_order % 2 == 0) {
    uint32_t runs0 = 0, g0 = 1;     // run count and runs per unit of the regular segments
    for (uint32_t idx : bulk_segs)
      if (dp.segs[idx].run_bytes >= T) {
        runs0 = dp.segs[idx].n_runs;
        g0 = runs_per_unit((uint32_t)((dp.segs[idx].run_bytes + T - 1) / T));
        break;
      }
    uint64_t upg = 0;               // units per group of g0 runs, over all regular segments
    for (uint32_t idx : bulk_segs) {
      const uint64_t tpr = (dp.segs[idx].run_bytes + T - 1) / T;
      if (runs0 == 0 || dp.segs[idx].run_bytes < T || dp.segs[idx].n_runs != runs0 ||
          runs_per_unit((uint32_t)tpr) != g0) {
        rest.push_back(idx);
        continue;
      }
      dp.gen_seg.push_back(idx);
      dp.gen_pre.push_back((uint32_t)upg);
      upg += g0 > 1 ? 1 : (tpr + kUnitTiles - 1) / kUnitTiles;
    }
    const uint64_t groups = (runs0 + g0 - 1) / g0;
    if (upg * groups < 0xffffffffull && upg < 0xffffffffull) {
      dp.gen_runs = runs0;
      dp.gen_group = g0;
      dp.gen_upr = (uint32_t)upg;
      dp.n_gen = upg * groups;
    } else {  // too many for 32-bit unit indices in the generator: everything on the host
      dp.gen_seg.clear(); dp.gen_pre.clear();
      rest = bulk_segs;
    }
  } else {
    rest = bulk_segs;
  }
  expand_units_on_host(&dp, rest, T, p->tuning.unit_order % 2 == 0);
  dp.n_bulk = dp.n_gen + dp.bulk_units.size();
  if (phase == EMOE_PHASE_KV) {  // block pairs of the head re-split, in launch order
    const KvPlan &kv = p->hp.kv;
    if (kv.head_split_changes && !kv.pair_old.empty())
      for (uint32_t rn = 0; rn < kv.d; ++rn)
        if (p->local_rank < 0 || (int)rn == p->local_rank)
          for (uint32_t hl = 0; hl < kv.hn; ++hl) p->reads_src[phase][kv.src_rank[rn * kv.hn + hl]] = true;
    std::vector<uint32_t> idx(kv.pair_old.size());
    for (uint32_t i = 0; i < idx.size(); ++i) idx[i] = i;
    if (kv_order(p) >= 2) {
      const std::vector<uint32_t> &key = kv_order(p) == 3 ? kv.pair_new : kv.pair_old;
      std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) { return key[a] < key[b]; });
    }
    p->pair_old.resize(idx.size());
    p->pair_new.resize(idx.size());
    for (size_t i = 0; i < idx.size(); ++i) {
      p->pair_old[i] = kv.pair_old[idx[i]];
      p->pair_new[i] = kv.pair_new[idx[i]];
    }
  }
}

// One launch set for the whole step: the three phases are independent of one another, so
// their segments can share a launch.  Ranks of the phases are renumbered into one pointer
// table (experts first, then attention, then KV); if they do not fit, the step falls back
// to phase-by-phase launches.
void build_merged(emoe_plan *p) {
  DevPhase &all = p->dev[3];
  all.segs.clear(); all.dsts.clear(); all.bulk_units.clear(); all.vec_units.clear();
  uint32_t ns = 0, nd = 0;
  for (int ph = 0; ph < 3; ++ph) {
    p->src_base[ph] = ns;
    p->dst_base[ph] = nd;
    ns += (uint32_t)p->hp.phase[ph].arena_old.size();
    nd += (uint32_t)p->hp.phase[ph].arena_new.size();
  }
  p->merged = ns <= EMOE_MAX_RANKS && nd <= EMOE_MAX_RANKS;
  if (!p->merged) return;
  all.gen_seg.clear(); all.gen_pre.clear();
  all.n_gen = 0; all.n_bulk = 0;
  size_t n_seg = 0, n_dst = 0, n_vec = 0, n_rest = 0;
  uint64_t n_bulk = 0;
  for (int ph = 0; ph < 3; ++ph) {
    const DevPhase &dp = p->dev[ph];
    p->merged_seg0[ph] = (uint32_t)n_seg;
    p->merged_unit0[ph] = n_bulk;          // the phase's generated units, then its host-built ones
    all.rest_off[ph] = n_rest;
    n_seg += dp.segs.size(); n_dst += dp.dsts.size();
    n_bulk += dp.n_bulk; n_vec += dp.vec_units.size(); n_rest += dp.bulk_units.size();
    all.n_gen += dp.n_gen;
  }
  if (n_bulk >= 0xffffffffull) { p->merged = false; return; }
  all.n_bulk = n_bulk;
  all.segs.resize(n_seg); all.dsts.resize(n_dst); all.vec_units.resize(n_vec);
  all.bulk_units.resize(n_rest);
  size_t i_seg = 0, i_dst = 0, i_bulk = 0, i_vec = 0;
  for (int ph = 0; ph < 3; ++ph) {
    const DevPhase &dp = p->dev[ph];
    const uint32_t seg0 = (uint32_t)i_seg, dst0 = (uint32_t)i_dst;
    for (const DevSeg &s0 : dp.segs) {
      DevSeg &s = all.segs[i_seg++];
      s = s0;
      s.src_rank += p->src_base[ph];
      s.dst_rank += p->dst_base[ph];
      s.dst_first += dst0;
    }
    for (const Dst &d0 : dp.dsts) {
      Dst &d = all.dsts[i_dst++];
      d = d0;
      d.rank += p->dst_base[ph];
    }
    for (const Unit &u0 : dp.bulk_units) { Unit &u = all.bulk_units[i_bulk++]; u = u0; u.seg += seg0; }
    for (const Unit &u0 : dp.vec_units) { Unit &u = all.vec_units[i_vec++]; u = u0; u.seg += seg0; }
  }
}

// Tables of the three phases (independent of one another: built on three threads when the
// plan is large enough to pay for them) and the merged set.  Throws std::bad_alloc.
void build_all_tables(emoe_plan *p) {
  uint64_t work = 0;
  for (int ph = 0; ph < 3; ++ph) work += p->hp.phase[ph].segs.size() + p->hp.phase[ph].bytes_moved / (1u << 20);
  if (work < 4096) {  // small plan: threads would cost more than they save
    for (int ph = 0; ph < 3; ++ph) build_tables(p, ph);
  } else {
    bool failed[3] = {false, false, false};
    std::thread th[2];
    for (int ph = 1; ph < 3; ++ph)
      th[ph - 1] = std::thread([p, ph, &failed] {
        try { build_tables(p, ph); } catch (...) { failed[ph] = true; }
      });
    try { build_tables(p, 0); } catch (...) { failed[0] = true; }
    for (std::thread &t : th) t.join();
    if (failed[0] || failed[1] || failed[2]) throw std::bad_alloc();
  }
  build_merged(p);
}

template <typename T>
cudaError_t upload(const std::vector<T> &v, T **d) {
  if (*d) { cudaFree(*d); *d = nullptr; }
  if (v.empty()) return cudaSuccess;
  cudaError_t e = cudaMalloc((void **)d, v.size() * sizeof(T));
  if (e != cudaSuccess) return e;
  return cudaMemcpy(*d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
}

emoe_status_t cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return EMOE_OK;
  (void)cudaGetLastError();
  return e == cudaErrorMemoryAllocation ? EMOE_ERR_OOM : EMOE_ERR_CUDA;
}

// Expands the regular unit table of phase `src_ph` into `out` on the device.
cudaError_t gen_units(const emoe_plan *p, int src_ph, const DevSeg *d_segs, uint32_t seg_offset, Unit *out) {
  const DevPhase &dp = p->dev[src_ph];
  uint32_t *d_idx = nullptr, *d_pre = nullptr;
  const size_t bytes = dp.gen_seg.size() * sizeof(uint32_t);
  cudaError_t e = cudaMalloc((void **)&d_idx, bytes);
  if (e == cudaSuccess) e = cudaMalloc((void **)&d_pre, bytes);
  if (e == cudaSuccess) e = cudaMemcpy(d_idx, dp.gen_seg.data(), bytes, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(d_pre, dp.gen_pre.data(), bytes, cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = launch_gen_units(d_segs, d_idx, d_pre, (uint32_t)dp.gen_seg.size(), dp.gen_runs, dp.gen_group,
                         dp.gen_upr, bulk_tile(p), kUnitTiles, seg_offset, out, nullptr);
  if (e == cudaSuccess) e = cudaStreamSynchronize(nullptr);
  cudaFree(d_idx);
  cudaFree(d_pre);
  return e;
}

emoe_status_t upload_phase(emoe_plan *p, int phase) {
  DevPhase &dp = p->dev[phase];
  cudaError_t e;
  if ((e = upload(dp.segs, &dp.d_segs)) != cudaSuccess) return cuda_status(e);
  if ((e = upload(dp.dsts, &dp.d_dsts)) != cudaSuccess) return cuda_status(e);
  if ((e = upload(dp.vec_units, &dp.d_vec_units)) != cudaSuccess) return cuda_status(e);
  // bulk unit table: generated part(s) written by a kernel, host-built part(s) copied after them
  if (dp.d_bulk_units) { cudaFree(dp.d_bulk_units); dp.d_bulk_units = nullptr; }
  if (dp.n_bulk == 0) return EMOE_OK;
  if ((e = cudaMalloc((void **)&dp.d_bulk_units, dp.n_bulk * sizeof(Unit))) != cudaSuccess) return cuda_status(e);
  auto copy_rest = [&](const Unit *host, uint64_t n, Unit *dev) {
    return n ? cudaMemcpy(dev, host, n * sizeof(Unit), cudaMemcpyHostToDevice) : cudaSuccess;
  };
  if (phase < 3) {
    if (dp.n_gen && (e = gen_units(p, phase, dp.d_segs, 0, dp.d_bulk_units)) != cudaSuccess) return cuda_status(e);
    return cuda_status(copy_rest(dp.bulk_units.data(), dp.bulk_units.size(), dp.d_bulk_units + dp.n_gen));
  }
  for (int q = 0; q < 3; ++q) {
    const DevPhase &dq = p->dev[q];
    Unit *at = dp.d_bulk_units + p->merged_unit0[q];
    if (dq.n_gen && (e = gen_units(p, q, dp.d_segs, p->merged_seg0[q], at)) != cudaSuccess) return cuda_status(e);
    e = copy_rest(dp.bulk_units.data() + dp.rest_off[q], dq.bulk_units.size(), at + dq.n_gen);
    if (e != cudaSuccess) return cuda_status(e);
  }
  return EMOE_OK;
}

void free_device(emoe_plan *p) {
  for (DevPhase &dp : p->dev) {
    cudaFree(dp.d_segs); cudaFree(dp.d_dsts); cudaFree(dp.d_bulk_units); cudaFree(dp.d_vec_units);
    dp.d_segs = nullptr; dp.d_dsts = nullptr; dp.d_bulk_units = dp.d_vec_units = nullptr;
  }
  cudaFree(p->d_pair_old); cudaFree(p->d_pair_new); cudaFree(p->d_status);
  p->d_pair_old = p->d_pair_new = nullptr; p->d_status = nullptr;
  for (cudaStream_t &sd : p->side) { if (sd) cudaStreamDestroy(sd); sd = nullptr; }
  if (p->ev_fork) cudaEventDestroy(p->ev_fork);
  if (p->ev_join) cudaEventDestroy(p->ev_join);
  p->ev_fork = p->ev_join = nullptr;
}

int ranks_of(const emoe_plan *p, int phase, int side) {
  if (phase == EMOE_PHASE_EXPERTS) return side == EMOE_SIDE_OLD ? p->hp.ep_old : p->hp.ep_new;
  if (side == EMOE_SIDE_OLD) return p->hp.tp_old;
  return phase == EMOE_PHASE_ATTN ? p->hp.tp_new * (int)p->hp.attn_replicas : p->hp.tp_new;
}

// Host-side argument checks of a reshard call; fills the by-value pointer table.
// *zero_copy (optional) is set when the phase changes nothing AND the caller passed, for every
// rank, the very arena it already has (dst[r] == src[r]): the paper's zero-copy case - the new
// configuration goes on using the memory in place and nothing is launched.
emoe_status_t check_arenas(const emoe_plan *p, int phase, const void *const *src, void *const *dst,
                           RankPtrs *out, bool *zero_copy = nullptr) {
  if (zero_copy) *zero_copy = false;
  if (!p || !src || !dst || p->inplace) return EMOE_ERR_INVALID_ARG;
  if (p->host_only) return EMOE_ERR_CUDA;
  // the plan's tables, counters and streams belong to the device it was made on
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) return EMOE_ERR_CUDA;
  const PhasePlan &pp = p->hp.phase[phase];
  const int ns = ranks_of(p, phase, EMOE_SIDE_OLD), nd = ranks_of(p, phase, EMOE_SIDE_NEW);
  std::memset(out, 0, sizeof(*out));
  if (zero_copy && pp.identity && ns == nd) {
    bool same = true;   // with a local rank set only that rank's arena is looked at
    for (int r = 0; r < ns; ++r)
      if (p->local_rank < 0 || r == p->local_rank)
        same = same && src[r] == dst[r] && (src[r] || !pp.arena_old[r]);
    if (same) { *zero_copy = true; return EMOE_OK; }
  }
  // With a local rank set, only that rank's destination arena and the source arenas its
  // work reads are needed; the other entries may be NULL and are never dereferenced.
  const bool local = p->local_rank >= 0;
  for (int r = 0; r < ns; ++r) {
    const bool needed = local ? p->reads_src[phase][r] : pp.arena_old[r] != 0;
    if (needed && !src[r]) return EMOE_ERR_INVALID_ARG;
    if ((uintptr_t)src[r] % 16) return EMOE_ERR_ALIGNMENT;
    out->src[r] = (const uint8_t *)src[r];
  }
  for (int r = 0; r < nd; ++r) {
    const bool needed = pp.arena_new[r] != 0 && (!local || r == p->local_rank);
    if (needed && !dst[r]) return EMOE_ERR_INVALID_ARG;
    if ((uintptr_t)dst[r] % 16) return EMOE_ERR_ALIGNMENT;
    out->dst[r] = needed ? (uint8_t *)dst[r] : nullptr;
  }
  for (int a = 0; a < ns; ++a)
    for (int b = 0; b < nd; ++b) {
      if (!src[a] || !out->dst[b]) continue;
      const uintptr_t s0 = (uintptr_t)src[a], s1 = s0 + pp.arena_old[a];
      const uintptr_t d0 = (uintptr_t)dst[b], d1 = d0 + pp.arena_new[b];
      if (s0 < d1 && d0 < s1) return EMOE_ERR_OVERLAP;
    }
  return EMOE_OK;
}

uint32_t bulk_budget(const emoe_plan *p) {
  if (p->tuning.max_ctas > 0) return (uint32_t)p->tuning.max_ctas;
  return kDefaultBulkCtas < (uint32_t)p->sm_count ? kDefaultBulkCtas : (uint32_t)p->sm_count;
}

uint32_t cta_budget(const emoe_plan *p) {
  return p->tuning.max_ctas > 0 ? (uint32_t)p->tuning.max_ctas : (uint32_t)p->sm_count;
}

// Launch configuration of the bulk kernel for a launch of `grid` CTAs.
BulkConfig bulk_config(const emoe_plan *p, uint32_t grid) {
  BulkConfig bc{bulk_tile(p), bulk_stages(p),
                p->tuning.bulk_hints > 0 ? (uint32_t)p->tuning.bulk_hints - 1 : kDefaultHints, 0, wait_ns(p)};
  if (p->tuning.bw_limit_gbs > 0 && grid > 0) {
    // The limit counts bytes read plus bytes written, so loads get half of it; spread over
    // the CTAs that run at the same time - the grid, or what fits the SMs when the grid is
    // larger - that is one tile per CTA every tile * CTAs / (limit / 2) ns.
    const size_t per_cta = bulk_smem_bytes(bc.tile_bytes, bc.stages) + 2048;
    const uint64_t fit = (uint64_t)p->sm_count * std::max<size_t>(1, (227 * 1024) / per_cta);
    const double ctas = (double)std::min<uint64_t>(grid, fit);
    const double ns = 2.0 * bc.tile_bytes * ctas / (double)p->tuning.bw_limit_gbs;
    bc.pace_ns = ns < 1.0 ? 1u : ns > 1e6 ? 1000000u : (uint32_t)ns;
  }
  return bc;
}

// The bulk launch of a table set.  Its work counter: the set's slots are used in turn; a
// launch that is being captured into a graph gets none (its CTAs take units round-robin),
// because a graph would keep its slot for as long as it lives.
emoe_status_t run_bulk(const emoe_plan *p, int set, const RankPtrs &ptrs, cudaStream_t st) {
  const DevPhase &dp = p->dev[set];
  if (dp.n_bulk == 0) return EMOE_OK;
  unsigned int *ctr = nullptr;
  if (p->tuning.unit_order < 2) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { (void)cudaGetLastError(); cs = cudaStreamCaptureStatusNone; }
    if (cs == cudaStreamCaptureStatusNone) {
      const uint32_t slot = p->launch_seq[set].fetch_add(1) % kCtrSlots;
      ctr = reinterpret_cast<unsigned int *>(p->d_status) + 1 + (set * kCtrSlots + slot) * 2;
    }
  }
  uint32_t grid = bulk_budget(p);
  if (grid > dp.n_bulk) grid = (uint32_t)dp.n_bulk;
  return cuda_status(launch_bulk_copy({dp.d_segs, dp.d_dsts, dp.d_bulk_units, (uint32_t)dp.n_bulk}, ptrs,
                                      bulk_config(p, grid), grid, p->d_status, ctr, st));
}

uint32_t vec_grid(const emoe_plan *p) {
  return p->tuning.max_ctas > 0 ? cta_budget(p) * 8 : 0xffffffffu;
}

emoe_status_t run_vec(const emoe_plan *p, int set, const RankPtrs &ptrs, cudaStream_t st) {
  const DevPhase &dp = p->dev[set];
  return cuda_status(launch_vec_copy({dp.d_segs, dp.d_dsts, dp.d_vec_units, (uint32_t)dp.vec_units.size()},
                                     ptrs, kVecTile, vec_grid(p), st));
}

// path = 3: the segments of a phase as driver copies - one (strided) device-to-device copy
// per segment and destination, which the driver hands to the GPU's copy engines: no SM, no
// shared memory is taken from a kernel that runs beside the reshard.  Only for comparison and
// for sharing the GPU: a replicated source is read once per destination, every segment is an
// API call, and the rate is the copy engines'.
emoe_status_t run_segments_by_copy_engine(const emoe_plan *p, int phase, const RankPtrs &ptrs, cudaStream_t st) {
  const PhasePlan &pp = p->hp.phase[phase];
  for (const Segment &s : pp.segs)
    for (uint32_t j = 0; j < s.n_dst; ++j) {
      const Dst &d = pp.dsts[s.dst_first + j];
      if (p->local_rank >= 0 && (int)d.rank != p->local_rank) continue;
      const uint8_t *src = ptrs.src[s.src_rank] + s.src_off;
      uint8_t *dst = ptrs.dst[d.rank] + d.off;
      // a strided copy takes pitches below 2 GiB; runs that are further apart go one by one
      const bool strided = s.n_runs > 1 && d.pitch < (1ull << 31) && s.src_pitch < (1ull << 31);
      cudaError_t e = cudaSuccess;
      if (strided) {
        e = cudaMemcpy2DAsync(dst, d.pitch, src, s.src_pitch, s.run_bytes, s.n_runs, cudaMemcpyDeviceToDevice, st);
      } else {
        for (uint32_t r = 0; e == cudaSuccess && r < s.n_runs; ++r)
          e = cudaMemcpyAsync(dst + (uint64_t)r * d.pitch, src + (uint64_t)r * s.src_pitch, s.run_bytes,
                              cudaMemcpyDeviceToDevice, st);
      }
      if (e != cudaSuccess) return cuda_status(e);
    }
  return EMOE_OK;
}

emoe_status_t run_segments(const emoe_plan *p, int phase, const RankPtrs &ptrs, cudaStream_t st) {
  if (p->tuning.path == 3 && phase < 3) return run_segments_by_copy_engine(p, phase, ptrs, st);
  const emoe_status_t rc = run_bulk(p, phase, ptrs, st);
  return rc != EMOE_OK ? rc : run_vec(p, phase, ptrs, st);
}

// Shape constants of the KV head re-split as the kernels take them.
KvTables kv_tables(const KvPlan &kv, const uint32_t *d_pair_old, const uint32_t *d_pair_new,
                   int local_rank = -1) {
  KvTables t{};
  t.dst_only = local_rank >= 0 ? (uint32_t)local_rank : 0xffffffffu;
  t.pair_old = d_pair_old;
  t.pair_new = d_pair_new;
  t.n_pairs = (uint32_t)kv.pair_old.size();
  t.n_lk = kv.n_layers * 2;
  t.block_tokens = kv.block_tokens;
  t.hkv = kv.d * kv.hn;
  t.hc = kv.hc;
  t.hn = kv.hn;
  t.head_bytes = (uint32_t)kv.head_bytes;
  t.nb_old = kv.nb_old;
  t.nb_new = kv.nb_new;
  t.use_map = kv.replicated ? 1u : 0u;
  if (kv.replicated)  // at most max(old ranks, new ranks) <= EMOE_MAX_RANKS slots
    for (size_t j = 0; j < kv.src_rank.size() && j < kKvMapMax; ++j) {
      t.map_rank[j] = kv.src_rank[j];
      t.map_head[j] = (uint8_t)kv.src_head[j];
    }
  return t;
}

void destroy_host_step(HostStep *hs);

emoe_status_t create_plan(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                          const emoe_config_t *new_cfg, uint32_t flags, emoe_plan_t **out,
                          uint64_t expert_scale_bytes = 0, uint32_t attn_replicas = 1);

// Chunk plans, streams and events of the pipelined host-buffer step.  Leaves p->hs null
// (the step then runs serially) when a layer slice of some arena is not 16-byte aligned.
emoe_status_t make_host_step(emoe_plan *p, const emoe_shape_t &shape, const emoe_config_t *old_cfg,
                             const emoe_config_t *new_cfg, uint32_t layout_flags) {
  const int L = shape.n_layers;
  for (int ph = 0; ph < 3; ++ph) {
    for (uint64_t b : p->hp.phase[ph].arena_old) if ((b / L) % 16) return EMOE_OK;
    for (uint64_t b : p->hp.phase[ph].arena_new) if ((b / L) % 16) return EMOE_OK;
  }
  HostStep *hs = new (std::nothrow) HostStep();
  if (!hs) return EMOE_ERR_OOM;
  // up to 32 chunks (single layers for most models): the pipeline's fill and drain - the
  // first copy-in and the last copy-out, which nothing overlaps - shrink with the chunk
  hs->lc = (L + 31) / 32;
  const int n_full = L / hs->lc, tail = L % hs->lc;
  hs->n_chunks = n_full + (tail ? 1 : 0);
  emoe_shape_t sh = shape;
  sh.n_layers = hs->lc;
  emoe_status_t st = create_plan(&sh, old_cfg, new_cfg, layout_flags, &hs->chunk, 0, p->hp.attn_replicas);
  if (st == EMOE_OK && tail) {
    sh.n_layers = tail;
    st = create_plan(&sh, old_cfg, new_cfg, layout_flags, &hs->tail, 0, p->hp.attn_replicas);
  }
  cudaError_t e = cudaSuccess;
  if (st == EMOE_OK) e = cudaStreamCreateWithFlags(&hs->s_in, cudaStreamNonBlocking);
  if (st == EMOE_OK && e == cudaSuccess) e = cudaStreamCreateWithFlags(&hs->s_out, cudaStreamNonBlocking);
  if (st == EMOE_OK && e == cudaSuccess) e = cudaEventCreateWithFlags(&hs->ev_start, cudaEventDisableTiming);
  if (st == EMOE_OK && e == cudaSuccess) e = cudaEventCreateWithFlags(&hs->ev_done, cudaEventDisableTiming);
  try {
    for (int i = 0; st == EMOE_OK && e == cudaSuccess && i < hs->n_chunks; ++i) {
      cudaEvent_t a = nullptr, b = nullptr;
      e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b, cudaEventDisableTiming);
      hs->ev_in.push_back(a);
      hs->ev_k.push_back(b);
    }
  } catch (const std::bad_alloc &) {
    st = EMOE_ERR_OOM;
  }
  if (st == EMOE_OK) st = cuda_status(e);
  if (st != EMOE_OK) { destroy_host_step(hs); return st; }
  p->hs = hs;
  return EMOE_OK;
}

void destroy_host_step(HostStep *hs) {
  if (!hs) return;
  emoe_plan_destroy(hs->chunk);
  emoe_plan_destroy(hs->tail);
  for (cudaEvent_t ev : hs->ev_in) if (ev) cudaEventDestroy(ev);
  for (cudaEvent_t ev : hs->ev_k) if (ev) cudaEventDestroy(ev);
  if (hs->ev_start) cudaEventDestroy(hs->ev_start);
  if (hs->ev_done) cudaEventDestroy(hs->ev_done);
  if (hs->s_in) cudaStreamDestroy(hs->s_in);
  if (hs->s_out) cudaStreamDestroy(hs->s_out);
  delete hs;
}

// Device side of a new plan: descriptor tables, status word and work counters, the side
// streams of the whole step.  On failure everything is freed again.
emoe_status_t finish_device_plan(emoe_plan *p) {
  cudaError_t e = cudaGetDevice(&p->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
  if (e == cudaSuccess) e = kernels_init();   // per device: the plan's device is current
  emoe_status_t st = cuda_status(e);
  for (int ph = 0; st == EMOE_OK && ph < kTableSets; ++ph) st = upload_phase(p, ph);
  if (st == EMOE_OK && p->hp.kv.head_split_changes) {
    cudaError_t e2 = upload(p->pair_old, &p->d_pair_old);
    if (e2 == cudaSuccess) e2 = upload(p->pair_new, &p->d_pair_new);
    st = cuda_status(e2);
  }
  if (st == EMOE_OK) {
    cudaError_t e3 = cudaMalloc((void **)&p->d_status, kStatusWords * sizeof(int));
    if (e3 == cudaSuccess) e3 = cudaMemset(p->d_status, 0, kStatusWords * sizeof(int));
    if (e3 == cudaSuccess) e3 = cudaDeviceGetStreamPriorityRange(&p->prio_least, &p->prio_greatest);
    if (e3 == cudaSuccess) e3 = cudaStreamCreateWithPriority(&p->side[0], cudaStreamNonBlocking, p->prio_least);
    if (e3 == cudaSuccess) e3 = cudaStreamCreateWithPriority(&p->side[1], cudaStreamNonBlocking, p->prio_greatest);
    if (e3 == cudaSuccess) e3 = cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming);
    if (e3 == cudaSuccess) e3 = cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming);
    st = cuda_status(e3);
  }
  if (st != EMOE_OK) free_device(p);
  return st;
}

emoe_status_t create_plan(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                          const emoe_config_t *new_cfg, uint32_t flags, emoe_plan_t **out,
                          uint64_t expert_scale_bytes, uint32_t attn_replicas) {
  if (!shape || !old_cfg || !new_cfg || !out) return EMOE_ERR_INVALID_ARG;
  if (expert_scale_bytes && (flags & EMOE_LAYOUT_FUSED_W13)) return EMOE_ERR_UNSUPPORTED;
  emoe_plan *p = new (std::nothrow) emoe_plan();
  if (!p) return EMOE_ERR_OOM;
  emoe_status_t st;
  try {
    st = build_host_plan(*shape, *old_cfg, *new_cfg, flags, expert_scale_bytes, attn_replicas, &p->hp);
    if (st == EMOE_OK) {
      build_all_tables(p);
    }
  } catch (const std::bad_alloc &) {
    st = EMOE_ERR_OOM;
  }
  if (st != EMOE_OK) { delete p; return st; }
  p->host_only = (flags & EMOE_PLAN_HOST_ONLY) != 0;
  if (!p->host_only) {
    st = finish_device_plan(p);
    // (an expert arena with a scale part is not layer-major: such a plan's host step stays serial)
    if (st == EMOE_OK && (flags & EMOE_PLAN_HOST_STEP) && !expert_scale_bytes) {
      st = make_host_step(p, *shape, old_cfg, new_cfg,
                          flags & (EMOE_LAYOUT_FUSED_W13 | EMOE_LAYOUT_KV_HEAD_MAJOR | EMOE_LAYOUT_FUSED_QKV));
      if (st != EMOE_OK) free_device(p);
    }
    if (st != EMOE_OK) { delete p; return st; }
  }
  *out = p;
  return EMOE_OK;
}

}  // namespace

emoe_status_t emoe::run_phase_once(const PhasePlan &pp, const RankPtrs &ptrs, cudaStream_t st) {
  emoe_plan tmp;
  tmp.host_only = false;
  emoe_status_t rc = EMOE_OK;
  try {
    tmp.hp.phase[0] = pp;
    build_tables(&tmp, 0);
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  cudaError_t e = cudaGetDevice(&tmp.device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&tmp.sm_count, cudaDevAttrMultiProcessorCount, tmp.device);
  if (e == cudaSuccess) e = kernels_init();
  rc = cuda_status(e);
  if (rc == EMOE_OK) rc = upload_phase(&tmp, 0);
  if (rc == EMOE_OK) {
    e = cudaMalloc((void **)&tmp.d_status, kStatusWords * sizeof(int));
    if (e == cudaSuccess) e = cudaMemsetAsync(tmp.d_status, 0, kStatusWords * sizeof(int), st);
    rc = cuda_status(e);
  }
  if (rc == EMOE_OK) rc = run_segments(&tmp, 0, ptrs, st);
  int status = 0;
  if (rc == EMOE_OK) {
    e = cudaMemcpyAsync(&status, tmp.d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    rc = cuda_status(e);
    if (rc == EMOE_OK && status != 0) rc = (emoe_status_t)status;
  } else {
    (void)cudaStreamSynchronize(st);
  }
  free_device(&tmp);
  return rc;
}

extern "C" {

emoe_status_t emoe_plan_create(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                               const emoe_config_t *new_cfg, uint32_t flags, emoe_plan_t **out) {
  TraceRange trace("emoe_plan_create");
  return create_plan(shape, old_cfg, new_cfg, flags, out);
}

emoe_status_t emoe_plan_create_ex(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                                  const emoe_config_t *new_cfg, uint32_t flags,
                                  const emoe_plan_options_t *options, emoe_plan_t **out) {
  uint64_t scale = 0;
  uint32_t replicas = 1;
  if (options) {
    if (options->expert_scale_bytes < 0 || options->attn_new_replicas < 0 ||
        options->attn_new_replicas > EMOE_MAX_RANKS)
      return EMOE_ERR_INVALID_ARG;
    for (int64_t r : options->reserved)
      if (r != 0) return EMOE_ERR_INVALID_ARG;
    scale = (uint64_t)options->expert_scale_bytes;
    if (options->attn_new_replicas > 1) replicas = (uint32_t)options->attn_new_replicas;
  }
  return create_plan(shape, old_cfg, new_cfg, flags, out, scale, replicas);
}

void emoe_plan_destroy(emoe_plan_t *p) {
  if (!p) return;
  destroy_host_step(p->hs);
  if (!p->host_only) free_device(p);
  delete p;
}

emoe_status_t emoe_reshard_experts(const emoe_plan_t *p, const void *const *src, void *const *dst,
                                   void *stream) {
  TraceRange trace("emoe_reshard_experts");
  RankPtrs ptrs;
  bool zero_copy = false;
  emoe_status_t st = check_arenas(p, EMOE_PHASE_EXPERTS, src, dst, &ptrs, &zero_copy);
  if (st != EMOE_OK || zero_copy) return st;
  return run_segments(p, EMOE_PHASE_EXPERTS, ptrs, (cudaStream_t)stream);
}

emoe_status_t emoe_reshard_attn(const emoe_plan_t *p, const void *const *src, void *const *dst,
                                void *stream) {
  TraceRange trace("emoe_reshard_attn");
  RankPtrs ptrs;
  bool zero_copy = false;
  emoe_status_t st = check_arenas(p, EMOE_PHASE_ATTN, src, dst, &ptrs, &zero_copy);
  if (st != EMOE_OK || zero_copy) return st;
  return run_segments(p, EMOE_PHASE_ATTN, ptrs, (cudaStream_t)stream);
}

int32_t emoe_plan_phase_is_identity(const emoe_plan_t *p, int32_t phase) {
  if (!p || phase < 0 || phase > 2 || p->inplace) return -1;
  return p->hp.phase[phase].identity ? 1 : 0;
}

emoe_status_t emoe_reshard_kv(const emoe_plan_t *p, const void *const *src, void *const *dst,
                              void *stream) {
  TraceRange trace("emoe_reshard_kv");
  RankPtrs ptrs;
  bool zero_copy = false;
  emoe_status_t st = check_arenas(p, EMOE_PHASE_KV, src, dst, &ptrs, &zero_copy);
  if (st != EMOE_OK || zero_copy) return st;
  if (!p->hp.kv.head_split_changes) return run_segments(p, EMOE_PHASE_KV, ptrs, (cudaStream_t)stream);
  const KvPlan &kv = p->hp.kv;
  KvTables t = kv_tables(kv, p->d_pair_old, p->d_pair_new, p->local_rank);
  const int mode = kv_mode(p);
  return cuda_status(launch_kv_copy(t, ptrs, mode, cta_budget(p), p->tuning.max_ctas <= 0, p->d_status,
                                    wait_ns(p), (cudaStream_t)stream));
}

emoe_status_t emoe_reshard_step(const emoe_plan_t *p, const void *const *const src[3],
                                void *const *const dst[3], void *stream) {
  TraceRange trace("emoe_reshard_step");
  if (!p || !src || !dst || p->inplace) return EMOE_ERR_INVALID_ARG;
  RankPtrs ph_ptrs[3];
  bool zero_copy[3], any_zero_copy = false;
  for (int ph = 0; ph < 3; ++ph) {  // every argument is checked before anything is enqueued
    if (!src[ph] || !dst[ph]) return EMOE_ERR_INVALID_ARG;
    const emoe_status_t st = check_arenas(p, ph, src[ph], dst[ph], &ph_ptrs[ph], &zero_copy[ph]);
    if (st != EMOE_OK) return st;
    any_zero_copy = any_zero_copy || zero_copy[ph];
  }
  cudaStream_t st = (cudaStream_t)stream;
  const KvPlan &kv = p->hp.kv;
  emoe_status_t rc = EMOE_OK;
  // Phase by phase: too many ranks for one pointer table, driver copies, or a phase that stays
  // where it is (zero-copy: that phase launches nothing).
  if (!p->merged || p->tuning.path == 3 || any_zero_copy) {
    for (int ph = 0; rc == EMOE_OK && ph < 3; ++ph)
      if (!zero_copy[ph]) rc = run_segments(p, ph, ph_ptrs[ph], st);
    if (rc == EMOE_OK && kv.head_split_changes) {
      KvTables t = kv_tables(kv, p->d_pair_old, p->d_pair_new, p->local_rank);
      rc = cuda_status(launch_kv_copy(t, ph_ptrs[2], kv_mode(p), cta_budget(p), p->tuning.max_ctas <= 0,
                                      p->d_status, wait_ns(p), st));
    }
    return rc;
  }
  RankPtrs all;
  std::memset(&all, 0, sizeof(all));
  for (int ph = 0; ph < 3; ++ph) {
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_OLD); ++r) all.src[p->src_base[ph] + r] = ph_ptrs[ph].src[r];
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_NEW); ++r) all.dst[p->dst_base[ph] + r] = ph_ptrs[ph].dst[r];
  }
  // Up to two launch sets: the ring kernel (long runs of all three phases), and the
  // register-copy work - short and strided runs plus the KV head re-split, as ONE kernel
  // when the re-split uses the direct copy (the default).  With both present the second
  // set runs beside the first on a stream of the plan's own, so that neither waits for
  // the other's ramp-up and tail.
  const DevPhase &dp = p->dev[3];
  const bool kv_work = kv.head_split_changes && !kv.pair_old.empty();
  const bool has_bulk = dp.n_bulk > 0, has_small = !dp.vec_units.empty() || kv_work;
  const bool fork = has_bulk && has_small && p->tuning.serial == 0 && p->side[0];
  cudaStream_t st2 = st;
  std::unique_lock<std::mutex> lock(p->fork_mu, std::defer_lock);
  if (fork) {
    int prio = 0;
    cudaError_t e = cudaStreamGetPriority(st, &prio);
    if (e != cudaSuccess) return cuda_status(e);
    st2 = (prio - p->prio_greatest) < (p->prio_least - prio) ? p->side[1] : p->side[0];
    lock.lock();
    e = cudaEventRecord(p->ev_fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st2, p->ev_fork, 0);
    if (e != cudaSuccess) return cuda_status(e);
  }
  rc = run_bulk(p, 3, all, st);
  if (rc == EMOE_OK && has_small) {
    KvTables t = kv_tables(kv, p->d_pair_old, p->d_pair_new, p->local_rank);
    if (kv_work && fused_kv(p, t)) {
      rc = cuda_status(launch_vec_kv_copy({dp.d_segs, dp.d_dsts, dp.d_vec_units, (uint32_t)dp.vec_units.size()},
                                          all, kVecTile, t, ph_ptrs[2],
                                          p->tuning.max_ctas > 0 ? cta_budget(p) * 8 : 0,
                                          p->tuning.max_ctas <= 0, st2));
    } else {
      rc = run_vec(p, 3, all, st2);
      if (rc == EMOE_OK && kv_work)
        rc = cuda_status(launch_kv_copy(t, ph_ptrs[2], kv_mode(p), cta_budget(p), p->tuning.max_ctas <= 0,
                                        p->d_status, wait_ns(p), st2));
    }
  }
  if (fork) {  // joined even after an error, so that the caller's stream never loses the side work
    cudaError_t e = cudaEventRecord(p->ev_join, st2);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, p->ev_join, 0);
    if (rc == EMOE_OK) rc = cuda_status(e);
  }
  return rc;
}

emoe_status_t emoe_plan_create_inplace(const emoe_shape_t *shape, int32_t ep_old,
                                       const int32_t *slot_off_old, const int32_t *slot_ids_old,
                                       int32_t ep_new, const int32_t *cap_new, const int32_t *want_off,
                                       const int32_t *want_ids, uint32_t flags, emoe_plan_t **out) {
  if (!shape || !out || (flags & ~EMOE_PLAN_HOST_ONLY)) return EMOE_ERR_INVALID_ARG;
  emoe_plan *p = new (std::nothrow) emoe_plan();
  if (!p) return EMOE_ERR_OOM;
  emoe_status_t st;
  try {
    st = build_inplace_expert_plan(*shape, ep_old, slot_off_old, slot_ids_old, ep_new, cap_new, want_off,
                                   want_ids, 0, &p->hp.phase[EMOE_PHASE_EXPERTS], &p->slot_new);
    if (st == EMOE_OK) {
      p->inplace = true;
      p->hp.shape = *shape;
      p->hp.ep_old = ep_old; p->hp.ep_new = ep_new;
      p->hp.tp_old = p->hp.tp_new = 0;       // no attention or KV phase in this kind of plan
      build_all_tables(p);
    }
  } catch (const std::bad_alloc &) {
    st = EMOE_ERR_OOM;
  }
  if (st != EMOE_OK) { delete p; return st; }
  p->host_only = (flags & EMOE_PLAN_HOST_ONLY) != 0;
  if (!p->host_only && (st = finish_device_plan(p)) != EMOE_OK) { delete p; return st; }
  *out = p;
  return EMOE_OK;
}

emoe_status_t emoe_plan_slot_table(const emoe_plan_t *p, int32_t rank, int32_t *out, int32_t cap,
                                   int32_t *n_slots) {
  if (!p || !p->inplace || rank < 0 || rank >= (int)p->slot_new.size() || (cap > 0 && !out))
    return EMOE_ERR_INVALID_ARG;
  const std::vector<int32_t> &t = p->slot_new[rank];
  if (n_slots) *n_slots = (int32_t)t.size();
  for (int32_t i = 0; i < cap && i < (int32_t)t.size(); ++i) out[i] = t[i];
  return EMOE_OK;
}

emoe_status_t emoe_reshard_experts_inplace(const emoe_plan_t *p, void *const *arenas, void *stream) {
  TraceRange trace("emoe_reshard_experts_inplace");
  if (!p || !arenas || !p->inplace) return EMOE_ERR_INVALID_ARG;
  if (p->host_only) return EMOE_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) return EMOE_ERR_CUDA;
  const PhasePlan &pp = p->hp.phase[EMOE_PHASE_EXPERTS];
  const int ns = p->hp.ep_old, nd = p->hp.ep_new, n = ns > nd ? ns : nd;
  RankPtrs ptrs;
  std::memset(&ptrs, 0, sizeof(ptrs));
  uint64_t bytes[EMOE_MAX_RANKS];
  const bool local = p->local_rank >= 0;
  for (int r = 0; r < n; ++r) {
    bytes[r] = r < ns ? pp.arena_old[r] : pp.arena_new[r];
    // with a local rank set only that rank's arena and the arenas it reads are needed
    const bool needed = local ? (r == p->local_rank || (r < ns && p->reads_src[EMOE_PHASE_EXPERTS][r]))
                              : bytes[r] != 0;
    if (needed && !arenas[r]) return EMOE_ERR_INVALID_ARG;
    if ((uintptr_t)arenas[r] % 16) return EMOE_ERR_ALIGNMENT;
    if (!needed || !arenas[r]) { bytes[r] = 0; continue; }
    if (r < ns) ptrs.src[r] = (const uint8_t *)arenas[r];
    if (r < nd) ptrs.dst[r] = (uint8_t *)arenas[r];
  }
  for (int a = 0; a < n; ++a)        // different devices' arenas must not intersect
    for (int b = a + 1; b < n; ++b) {
      const uintptr_t a0 = (uintptr_t)arenas[a], a1 = a0 + bytes[a];
      const uintptr_t b0 = (uintptr_t)arenas[b], b1 = b0 + bytes[b];
      if (bytes[a] && bytes[b] && a0 < b1 && b0 < a1) return EMOE_ERR_OVERLAP;
    }
  return run_segments(p, EMOE_PHASE_EXPERTS, ptrs, (cudaStream_t)stream);
}

emoe_status_t emoe_reshard_kv_static(const emoe_plan_t *p, const void *const *src, void *const *dst,
                                     void *stream) {
  TraceRange trace("emoe_reshard_kv_static");
  if (!p || !src || !dst || p->inplace) return EMOE_ERR_INVALID_ARG;
  const KvPlan &kv = p->hp.kv;
  // this entry point only has the token-major pair kernel: whole blocks (TP kept) are
  // layout-agnostic, a head re-split of head-major blocks is not
  if (kv.head_major && kv.c != kv.d) return EMOE_ERR_UNSUPPORTED;
  const std::vector<uint32_t> *pair_old = &kv.pair_old, *pair_new = &kv.pair_new;
  if (pair_old->size() > EMOE_STATIC_KV_MAX_PAIRS) return EMOE_ERR_TOO_LARGE;
  // the same argument checks as emoe_reshard_kv, but a host-only plan is welcome here.  With
  // a local rank set only that rank's destination and the old ranks it reads are needed.
  const PhasePlan &pp = p->hp.phase[EMOE_PHASE_KV];
  const bool local = p->local_rank >= 0;
  RankPtrs ptrs;
  std::memset(&ptrs, 0, sizeof(ptrs));
  for (int r = 0; r < p->hp.tp_old; ++r) {
    const bool needed = local ? p->reads_src[EMOE_PHASE_KV][r] : pp.arena_old[r] != 0;
    if (needed && !src[r]) return EMOE_ERR_INVALID_ARG;
    if ((uintptr_t)src[r] % 16) return EMOE_ERR_ALIGNMENT;
    ptrs.src[r] = (const uint8_t *)src[r];
  }
  for (int r = 0; r < p->hp.tp_new; ++r) {
    const bool needed = pp.arena_new[r] != 0 && (!local || r == p->local_rank);
    if (needed && !dst[r]) return EMOE_ERR_INVALID_ARG;
    if ((uintptr_t)dst[r] % 16) return EMOE_ERR_ALIGNMENT;
    ptrs.dst[r] = needed ? (uint8_t *)dst[r] : nullptr;
  }
  for (int a = 0; a < p->hp.tp_old; ++a)
    for (int b = 0; b < p->hp.tp_new; ++b) {
      if (!ptrs.src[a] || !ptrs.dst[b]) continue;
      const uintptr_t s0 = (uintptr_t)src[a], s1 = s0 + pp.arena_old[a];
      const uintptr_t d0 = (uintptr_t)dst[b], d1 = d0 + pp.arena_new[b];
      if (s0 < d1 && d0 < s1) return EMOE_ERR_OVERLAP;
    }
  KvTables t = kv_tables(kv, nullptr, nullptr, p->local_rank);
  return launch_kv_copy_static(t, pair_old->data(), pair_new->data(), ptrs, (cudaStream_t)stream);
}

}  // extern "C"

namespace {

// Chunk by chunk: copy the layers' slices of every old arena in (stream s_in), run the
// three phases on them (caller's stream), copy the slices of every new arena out (s_out).
// The three streams run concurrently, so copy-in of chunk i+1, kernels of chunk i and
// copy-out of chunk i-1 overlap and both directions of the host link stay busy.
emoe_status_t step_host_pipelined(const emoe_plan *p, const void *const *const h_src[3],
                                  void *const *const h_dst[3], void *const *const d_src[3],
                                  void *const *const d_dst[3], cudaStream_t st) {
  HostStep *hs = p->hs;
  const int L = p->hp.shape.n_layers;
  for (int ph = 0; ph < 3; ++ph) {
    if (!h_src[ph] || !h_dst[ph] || !d_src[ph] || !d_dst[ph]) return EMOE_ERR_INVALID_ARG;
    const PhasePlan &pp = p->hp.phase[ph];
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_OLD); ++r)
      if (pp.arena_old[r] && (!h_src[ph][r] || !d_src[ph][r])) return EMOE_ERR_INVALID_ARG;
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_NEW); ++r)
      if (pp.arena_new[r] && (!h_dst[ph][r] || !d_dst[ph][r])) return EMOE_ERR_INVALID_ARG;
  }
  cudaError_t e = cudaEventRecord(hs->ev_start, st);  // copies start after the stream's earlier work
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hs->s_in, hs->ev_start, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hs->s_out, hs->ev_start, 0);
  if (e != cudaSuccess) return cuda_status(e);
  const void *sp[3][EMOE_MAX_RANKS];
  void *dp[3][EMOE_MAX_RANKS];
  for (int ci = 0; ci < hs->n_chunks; ++ci) {
    const int l0 = ci * hs->lc, n = L - l0 < hs->lc ? L - l0 : hs->lc;
    const emoe_plan *sub = n == hs->lc ? hs->chunk : hs->tail;
    for (int ph = 0; ph < 3; ++ph) {
      const PhasePlan &pp = p->hp.phase[ph];
      for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_OLD); ++r) {
        const uint64_t lb = pp.arena_old[r] / L;
        sp[ph][r] = (const uint8_t *)d_src[ph][r] + l0 * lb;
        if (!lb) continue;
        e = cudaMemcpyAsync((uint8_t *)d_src[ph][r] + l0 * lb, (const uint8_t *)h_src[ph][r] + l0 * lb,
                            n * lb, cudaMemcpyHostToDevice, hs->s_in);
        if (e != cudaSuccess) return cuda_status(e);
      }
      for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_NEW); ++r)
        dp[ph][r] = (uint8_t *)d_dst[ph][r] + l0 * (pp.arena_new[r] / L);
    }
    e = cudaEventRecord(hs->ev_in[ci], hs->s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, hs->ev_in[ci], 0);
    if (e != cudaSuccess) return cuda_status(e);
    const void *const *sps[3] = {sp[0], sp[1], sp[2]};
    void *const *dps[3] = {dp[0], dp[1], dp[2]};
    const emoe_status_t rc = emoe_reshard_step(sub, sps, dps, st);
    if (rc != EMOE_OK) return rc;
    e = cudaEventRecord(hs->ev_k[ci], st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(hs->s_out, hs->ev_k[ci], 0);
    if (e != cudaSuccess) return cuda_status(e);
    for (int ph = 0; ph < 3; ++ph) {
      const PhasePlan &pp = p->hp.phase[ph];
      for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_NEW); ++r) {
        const uint64_t lb = pp.arena_new[r] / L;
        if (!lb) continue;
        e = cudaMemcpyAsync((uint8_t *)h_dst[ph][r] + l0 * lb, (const uint8_t *)d_dst[ph][r] + l0 * lb,
                            n * lb, cudaMemcpyDeviceToHost, hs->s_out);
        if (e != cudaSuccess) return cuda_status(e);
      }
    }
  }
  e = cudaEventRecord(hs->ev_done, hs->s_out);  // the caller's stream ends after the last copy-out
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, hs->ev_done, 0);
  return cuda_status(e);
}

}  // namespace

extern "C" {

emoe_status_t emoe_reshard_step_host(const emoe_plan_t *p, const void *const *const h_src[3],
                                     void *const *const h_dst[3], void *const *const d_src[3],
                                     void *const *const d_dst[3], void *stream) {
  TraceRange trace("emoe_reshard_step_host");
  if (!p || !h_src || !h_dst || !d_src || !d_dst || p->inplace) return EMOE_ERR_INVALID_ARG;
  if (p->host_only) return EMOE_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  if (p->hs) return step_host_pipelined(p, h_src, h_dst, d_src, d_dst, st);
  for (int ph = 0; ph < 3; ++ph) {
    if (!h_src[ph] || !h_dst[ph] || !d_src[ph] || !d_dst[ph]) return EMOE_ERR_INVALID_ARG;
    const PhasePlan &pp = p->hp.phase[ph];
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_OLD); ++r) {
      if (!pp.arena_old[r]) continue;
      if (!h_src[ph][r] || !d_src[ph][r]) return EMOE_ERR_INVALID_ARG;
      cudaError_t e = cudaMemcpyAsync(d_src[ph][r], h_src[ph][r], pp.arena_old[r],
                                      cudaMemcpyHostToDevice, st);
      if (e != cudaSuccess) return cuda_status(e);
    }
  }
  emoe_status_t rc = emoe_reshard_experts(p, (const void *const *)d_src[0], d_dst[0], stream);
  if (rc == EMOE_OK) rc = emoe_reshard_attn(p, (const void *const *)d_src[1], d_dst[1], stream);
  if (rc == EMOE_OK) rc = emoe_reshard_kv(p, (const void *const *)d_src[2], d_dst[2], stream);
  if (rc != EMOE_OK) return rc;
  for (int ph = 0; ph < 3; ++ph) {
    const PhasePlan &pp = p->hp.phase[ph];
    for (int r = 0; r < ranks_of(p, ph, EMOE_SIDE_NEW); ++r) {
      if (!pp.arena_new[r]) continue;
      if (!h_dst[ph][r]) return EMOE_ERR_INVALID_ARG;
      cudaError_t e = cudaMemcpyAsync(h_dst[ph][r], d_dst[ph][r], pp.arena_new[r],
                                      cudaMemcpyDeviceToHost, st);
      if (e != cudaSuccess) return cuda_status(e);
    }
  }
  return EMOE_OK;
}

emoe_status_t emoe_plan_num_ranks(const emoe_plan_t *p, int phase, int side, int32_t *n) {
  if (!p || !n || phase < 0 || phase > 2 || side < 0 || side > 1) return EMOE_ERR_INVALID_ARG;
  *n = ranks_of(p, phase, side);
  return EMOE_OK;
}

emoe_status_t emoe_plan_arena_bytes(const emoe_plan_t *p, int phase, int side, int rank,
                                    uint64_t *bytes) {
  if (!p || !bytes || phase < 0 || phase > 2 || side < 0 || side > 1) return EMOE_ERR_INVALID_ARG;
  if (rank < 0 || rank >= ranks_of(p, phase, side)) return EMOE_ERR_INVALID_ARG;
  const PhasePlan &pp = p->hp.phase[phase];
  *bytes = side == EMOE_SIDE_OLD ? pp.arena_old[rank] : pp.arena_new[rank];
  return EMOE_OK;
}

emoe_status_t emoe_plan_stats(const emoe_plan_t *p, int phase, uint64_t *bytes_moved,
                              uint64_t *bytes_read, uint64_t *n_segments) {
  if (!p || phase < 0 || phase > 2) return EMOE_ERR_INVALID_ARG;
  const PhasePlan &pp = p->hp.phase[phase];
  if (bytes_moved) *bytes_moved = pp.bytes_moved;
  if (bytes_read) *bytes_read = pp.bytes_read;
  if (n_segments) {
    *n_segments = pp.segs.size();
    if (phase == EMOE_PHASE_KV && p->hp.kv.head_split_changes) *n_segments = p->hp.kv.pair_old.size();
  }
  return EMOE_OK;
}

emoe_status_t emoe_plan_num_launches(const emoe_plan_t *p, int phase, int32_t *n) {
  if (!p || !n || phase < 0 || phase > EMOE_PHASE_STEP) return EMOE_ERR_INVALID_ARG;
  if (p->tuning.path == 3) {  // driver copies: the only kernel left is a KV head re-split
    const bool kv_here = phase == EMOE_PHASE_KV || phase == EMOE_PHASE_STEP;
    *n = kv_here && p->hp.kv.head_split_changes && !p->hp.kv.pair_old.empty() ? 1 : 0;
    return EMOE_OK;
  }
  if (phase == EMOE_PHASE_STEP) {  // launches of one emoe_reshard_step call
    const int kv_pairs = p->hp.kv.head_split_changes && !p->hp.kv.pair_old.empty() ? 1 : 0;
    int k = 0;
    if (p->merged) {
      const int vec = p->dev[3].vec_units.empty() ? 0 : 1;
      k = (p->dev[3].n_bulk ? 1 : 0);
      // the vector work and a direct KV head re-split share one kernel
      const KvTables t = kv_tables(p->hp.kv, nullptr, nullptr, p->local_rank);
      k += kv_pairs && fused_kv(p, t) ? 1 : vec + kv_pairs;
    } else {
      for (int ph = 0; ph < 3; ++ph)
        k += (p->dev[ph].n_bulk ? 1 : 0) + (p->dev[ph].vec_units.empty() ? 0 : 1);
      k += kv_pairs;
    }
    *n = k;
    return EMOE_OK;
  }
  if (phase == EMOE_PHASE_KV && p->hp.kv.head_split_changes) {
    *n = p->hp.kv.pair_old.empty() ? 0 : 1;
    return EMOE_OK;
  }
  *n = (p->dev[phase].n_bulk ? 1 : 0) + (p->dev[phase].vec_units.empty() ? 0 : 1);
  return EMOE_OK;
}

emoe_status_t emoe_plan_launch_work(const emoe_plan_t *p, int phase, uint64_t *ring_units,
                                    uint64_t *vector_units, uint64_t *kv_tiles) {
  if (!p || phase < 0 || phase > EMOE_PHASE_STEP) return EMOE_ERR_INVALID_ARG;
  const bool kv_here = (phase == EMOE_PHASE_KV || phase == EMOE_PHASE_STEP) && p->hp.kv.head_split_changes;
  uint64_t ring = 0, vec = 0;
  if (phase == EMOE_PHASE_STEP && !p->merged) {
    for (int ph = 0; ph < 3; ++ph) { ring += p->dev[ph].n_bulk; vec += p->dev[ph].vec_units.size(); }
  } else {
    ring = p->dev[phase].n_bulk;
    vec = p->dev[phase].vec_units.size();
  }
  if (ring_units) *ring_units = ring;
  if (vector_units) *vector_units = vec;
  if (kv_tiles) *kv_tiles = kv_here ? (uint64_t)p->hp.kv.pair_old.size() * p->hp.kv.n_layers * 2 : 0;
  return EMOE_OK;
}

emoe_status_t emoe_plan_segments(const emoe_plan_t *p, int phase, emoe_segment_t *out, uint64_t cap,
                                 uint64_t *n) {
  if (!p || !n || phase < 0 || phase > 2 || (cap && !out)) return EMOE_ERR_INVALID_ARG;
  try {
    std::vector<emoe_segment_t> v;
    export_segments(p->hp, phase, &v);
    *n = v.size();
    const uint64_t k = v.size() < cap ? v.size() : cap;
    if (k) std::memcpy(out, v.data(), k * sizeof(emoe_segment_t));
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}

emoe_status_t emoe_plan_validate(const emoe_plan_t *p, int32_t *bad_phase, uint64_t *bad_segment) {
  if (!p) return EMOE_ERR_INVALID_ARG;
  try {
    for (int ph = 0; ph < 3; ++ph) {
      if (p->inplace && ph != EMOE_PHASE_EXPERTS) continue;
      std::vector<emoe_segment_t> v;
      export_segments(p->hp, ph, &v);
      const PhasePlan &pp = p->hp.phase[ph];
      // weights must fill their new arenas exactly; not so the KV phase (unmapped blocks), the
      // in-place step (kept slots) and expert arenas with the gap before their scale part
      const bool tile = ph != EMOE_PHASE_KV && !p->inplace &&
                        !(ph == EMOE_PHASE_EXPERTS && p->hp.expert_scale_bytes);
      const emoe_status_t st = emoe_segments_validate(v.data(), v.size(), pp.arena_old.data(),
                                                      (int32_t)pp.arena_old.size(), pp.arena_new.data(),
                                                      (int32_t)pp.arena_new.size(), tile ? 1 : 0, bad_segment);
      if (st != EMOE_OK) {
        if (bad_phase) *bad_phase = ph;
        return st;
      }
    }
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}

emoe_status_t emoe_plan_device_status(const emoe_plan_t *p, int32_t *status) {
  if (!p || !status) return EMOE_ERR_INVALID_ARG;
  if (p->host_only) return EMOE_ERR_CUDA;
  int v = 0;
  cudaError_t e = cudaMemcpy(&v, p->d_status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_status(e);
  if (p->hs && v == 0) {  // the chunk plans of the pipelined host step have status words of their own
    int32_t sv = 0;
    for (const emoe_plan *sub : {p->hs->chunk, p->hs->tail})
      if (sub && v == 0 && emoe_plan_device_status(sub, &sv) == EMOE_OK) v = sv;
  }
  *status = v;
  return EMOE_OK;
}

emoe_status_t emoe_plan_clear_device_status(emoe_plan_t *p) {
  if (!p) return EMOE_ERR_INVALID_ARG;
  if (p->host_only) return EMOE_ERR_CUDA;
  if (cudaMemset(p->d_status, 0, sizeof(int)) != cudaSuccess) return cuda_status(cudaGetLastError());
  if (p->hs)
    for (emoe_plan *sub : {p->hs->chunk, p->hs->tail})
      if (sub) {
        const emoe_status_t rc = emoe_plan_clear_device_status(sub);
        if (rc != EMOE_OK) return rc;
      }
  return EMOE_OK;
}

emoe_status_t emoe_plan_set_tuning(emoe_plan_t *p, const emoe_tuning_t *t) {
  if (!p || !t) return EMOE_ERR_INVALID_ARG;
  if (t->max_ctas < 0 || t->bulk_tile_bytes < 0 || t->bulk_stages < 0 || t->path < 0 ||
      t->path > 3 || t->kv_mode < 0 || t->kv_mode > 4 || t->bulk_hints < 0 ||
      t->bulk_hints > 4 || t->kv_order < 0 || t->kv_order > 3 || t->unit_order < 0 ||
      t->unit_order > 3 || t->wait_limit_us < -1 || t->bw_limit_gbs < 0 || t->bulk_min_run < 0 ||
      t->serial < 0 || t->serial > 2)
    return EMOE_ERR_INVALID_ARG;
  if (t->bulk_tile_bytes && (t->bulk_tile_bytes % 128 || t->bulk_tile_bytes < 1024))
    return EMOE_ERR_INVALID_ARG;
  if (t->bulk_min_run && t->bulk_min_run % 16) return EMOE_ERR_INVALID_ARG;
  const uint32_t tile = t->bulk_tile_bytes ? t->bulk_tile_bytes : kDefaultBulkTile;
  const uint32_t stages = t->bulk_stages ? t->bulk_stages : kDefaultBulkStages;
  if (stages < 2 || stages > 16 || bulk_smem_bytes(tile, stages) > bulk_smem_limit())
    return EMOE_ERR_INVALID_ARG;
  if (p->hs)
    for (emoe_plan *sub : {p->hs->chunk, p->hs->tail})
      if (sub) {
        const emoe_status_t rc = emoe_plan_set_tuning(sub, t);
        if (rc != EMOE_OK) return rc;
      }
  p->tuning = *t;
  emoe_status_t st = EMOE_OK;
  try {
    build_all_tables(p);
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  if (!p->host_only) {
    if (cudaDeviceSynchronize() != cudaSuccess) return EMOE_ERR_CUDA;
    for (int ph = 0; st == EMOE_OK && ph < kTableSets; ++ph) st = upload_phase(p, ph);
    if (st == EMOE_OK && p->hp.kv.head_split_changes) {
      cudaError_t e2 = upload(p->pair_old, &p->d_pair_old);
      if (e2 == cudaSuccess) e2 = upload(p->pair_new, &p->d_pair_new);
      st = cuda_status(e2);
    }
  }
  return st;
}

emoe_status_t emoe_plan_set_local_rank(emoe_plan_t *p, int32_t rank) {
  if (!p || rank < -1 || rank >= EMOE_MAX_RANKS) return EMOE_ERR_INVALID_ARG;
  if (p->hs) return EMOE_ERR_UNSUPPORTED;  // the pipelined host step works on whole steps
  p->local_rank = rank;
  emoe_status_t st = EMOE_OK;
  try {
    build_all_tables(p);
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  if (!p->host_only) {
    if (cudaDeviceSynchronize() != cudaSuccess) return EMOE_ERR_CUDA;
    for (int ph = 0; st == EMOE_OK && ph < kTableSets; ++ph) st = upload_phase(p, ph);
  }
  return st;
}

emoe_status_t emoe_ipc_export(const void *device_ptr, void *handle_out, uint64_t *offset_out) {
  if (!device_ptr || !handle_out || !offset_out) return EMOE_ERR_INVALID_ARG;
  // the handle names the whole allocation: report where inside it the pointer lies
  using GetRangeFn = CUresult (*)(CUdeviceptr *, size_t *, CUdeviceptr);
  static GetRangeFn get_range = [] {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      f = nullptr;
    }
    return reinterpret_cast<GetRangeFn>(f);
  }();
  if (!get_range) return EMOE_ERR_UNSUPPORTED;
  CUdeviceptr base = 0;
  size_t size = 0;
  if (get_range(&base, &size, (CUdeviceptr)(uintptr_t)device_ptr) != CUDA_SUCCESS) return EMOE_ERR_CUDA;
  cudaIpcMemHandle_t h;
  if (cudaIpcGetMemHandle(&h, reinterpret_cast<void *>(base)) != cudaSuccess) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  static_assert(sizeof(h) == EMOE_IPC_HANDLE_BYTES, "handle size");
  std::memcpy(handle_out, &h, sizeof(h));
  *offset_out = (uint64_t)((uintptr_t)device_ptr - (uintptr_t)base);
  return EMOE_OK;
}

emoe_status_t emoe_ipc_open(const void *handle, void **base_out) {
  if (!handle || !base_out) return EMOE_ERR_INVALID_ARG;
  cudaIpcMemHandle_t h;
  std::memcpy(&h, handle, sizeof(h));
  void *base = nullptr;
  if (cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  *base_out = base;
  return EMOE_OK;
}

emoe_status_t emoe_ipc_close(void *base) {
  if (!base) return EMOE_OK;
  if (cudaIpcCloseMemHandle(base) != cudaSuccess) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  return EMOE_OK;
}

const char *emoe_strerror(emoe_status_t s) {
  switch (s) {
    case EMOE_OK: return "ok";
    case EMOE_ERR_INVALID_ARG: return "invalid argument";
    case EMOE_ERR_SHAPE: return "invalid model shape or TP degree does not divide the head counts";
    case EMOE_ERR_PLACEMENT: return "invalid expert placement";
    case EMOE_ERR_BLOCK_TABLE: return "invalid KV block table";
    case EMOE_ERR_ALIGNMENT: return "arena base pointer is not 16-byte aligned";
    case EMOE_ERR_OVERLAP: return "source and destination arenas overlap";
    case EMOE_ERR_OOM: return "out of memory";
    case EMOE_ERR_CUDA: return "CUDA error, or a host-only plan was asked to run";
    case EMOE_ERR_UNSUPPORTED: return "unsupported configuration";
    case EMOE_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case EMOE_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of this entry point";
    case EMOE_ERR_PLAN_CHECK: return "a copy run leaves its arena or two runs write the same byte";
  }
  return "unknown status";
}

}  // extern "C"
