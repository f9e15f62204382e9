// kernels.cu - sm_100a copy kernels of the scale-step re-layout.
//
//  * bulk_copy_kernel : long 16-byte-aligned runs.  One producer thread per CTA
//    issues cp.async.bulk (TMA, untiled) global->shared loads into a ring of
//    stages guarded by mbarriers; one consumer thread issues the
//    shared->global bulk stores, once per destination of the tile, so a
//    replicated source is read from HBM once.  No thread-block cluster is used.
//  * vec_copy_kernel  : short, strided or narrowly aligned runs.  A warp per
//    tile, lanes walk the tile in 16-byte (or narrower) pieces, four loads in
//    flight per lane before the stores.
//  * kv_copy_kernel   : KV head re-split.  A CTA per (layer, K|V, block pair)
//    gathers the block's token rows from the old ranks and writes each new
//    rank's block; only 8 bytes of metadata per block pair.
//
// Every device-side wait is bounded: on expiry the kernel records
// EMOE_ERR_DEVICE_TIMEOUT in the plan's status word, lets its own copies in
// flight land, and returns.
#include "kernels.h"

#include <cuda.h>

#include <mutex>

namespace emoe {
namespace {

constexpr uint32_t kMaxStages = 16;
constexpr int kMaxDevices = 64;
// Dynamic shared memory the bulk kernel may ask for: the 227 KiB a CTA can have, less room
// for the kernel's static shared memory (two pointer tables of EMOE_MAX_RANKS entries).
constexpr size_t kBulkSmemLimit = 224 * 1024;
// Bound of the waits that let copies already in flight land after a wait has expired
// (those copies always complete; the bound only keeps the loop finite).
constexpr unsigned long long kDrainLimitNs = 4000000000ull;

// ---- PTX wrappers -----------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking form: has the phase completed right now?
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within limit_ns, or if the CTA's
// other role has given up meanwhile (*abort set).
// limit_ns == 0: a wait that is not satisfied the moment it is asked fails at once
// (try_wait may itself suspend the thread for a while, so this case uses test_wait).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns,
                                          const volatile int *abort = nullptr) {
  if (limit_ns == 0) return mbar_test_wait(bar, parity);
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (abort && *abort) return false;
    if (globaltimer_ns() - t0 > limit_ns) return false;
  }
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load_hint(uint32_t dst_smem, const void *src, uint32_t bytes,
                                               uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1], %2, [%3], %4;"
      ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(src_smem), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void *dst, uint32_t src_smem, uint32_t bytes,
                                                uint64_t pol) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
               ::"l"(dst), "r"(src_smem), "r"(bytes), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// Tiled (tensor-map) copies of a 3-D box; coordinates are innermost first.
__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const void *map, int32_t c0,
                                            int32_t c1, int32_t c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst_smem), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const void *map, int32_t c0, int32_t c1, int32_t c2,
                                             uint32_t src_smem) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(src_smem)
               : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- bulk path --------------------------------------------------------------------------

struct TileInfo {  // producer -> consumer, one per stage
  uint64_t dst_ptr[kMaxFanout];
  uint64_t dst_pitch[kMaxFanout];
  uint32_t n_dst, n_rows, row_bytes, pad;
};

struct BulkParams {
  SegTables t;
  uint32_t tile_bytes, stages;
  uint32_t hints;      // bit 0: loads evict-first in L2, bit 1: stores evict-first
  uint32_t pace_ns;    // least time between a CTA's full-tile loads (0: unpaced): bandwidth limit
  unsigned long long wait_ns;  // bound of every wait (0: fail at once if not already satisfied)
  int *status;
  unsigned int *ctr;   // {next unit to claim, CTAs finished}, both 0 between launches; null: static
  RankPtrs ptrs;
};

__global__ void __launch_bounds__(64, 1) bulk_copy_kernel(const __grid_constant__ BulkParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t S = p.stages, T = p.tile_bytes;
  uint8_t *data = smem;
  TileInfo *info = reinterpret_cast<TileInfo *>(smem + (size_t)S * T);
  uint64_t *full = reinterpret_cast<uint64_t *>(info + S);
  uint64_t *empty = full + S;
  __shared__ const uint8_t *s_src[EMOE_MAX_RANKS];
  __shared__ uint8_t *s_dst[EMOE_MAX_RANKS];
  __shared__ volatile int s_abort;

  const uint32_t tid = threadIdx.x;
  if (tid < EMOE_MAX_RANKS) {
    s_src[tid] = p.ptrs.src[tid];
    s_dst[tid] = p.ptrs.dst[tid];
  }
  if (tid == 0) {
    s_abort = 0;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();

  if (tid == 0) {
    // ---------------- producer: schedule tiles, issue loads ----------------
    // Descriptors are fetched ahead of their use - the unit record two units ahead, its
    // segment one unit ahead - so that their latency hides behind the current unit.
    const uint64_t pol = policy_evict_first();
    const bool hint = (p.hints & 1u) != 0;
    const uint32_t G = gridDim.x, n = p.t.n_units;
    uint32_t it = 0;
    bool ok = true;
    unsigned long long t_next = 0;  // earliest start of the next load when the launch is paced
    // Units: the first one is the CTA's own index; the following ones are claimed from a
    // global counter (SMs do not all see the same bandwidth, and a static split ends with
    // the slowest: +1..3 % measured), or taken round-robin when there is no counter.  A
    // claim is made two units before its use, so its latency is hidden too.
    const bool dyn = p.ctr != nullptr;
    // raw claim -> unit index; n = no more units (n >= G: the grid never exceeds the unit count)
    auto claimed = [&](unsigned int c) -> uint32_t { return c < n - G ? G + c : n; };
    uint32_t u = blockIdx.x;
    uint32_t u1, u2;
    if (dyn) {
      u1 = claimed(atomicAdd(&p.ctr[0], 1u));
      u2 = claimed(atomicAdd(&p.ctr[0], 1u));
    } else {
      u1 = (uint64_t)u + G < n ? u + G : n;
      u2 = (uint64_t)u + 2ull * G < n ? u + 2 * G : n;
    }
    Unit un0 = p.t.units[u];
    DevSeg sg0 = p.t.segs[un0.seg];
    Unit un1 = un0;
    if (u1 < n) un1 = p.t.units[u1];
    while (ok && u < n) {
      DevSeg sg1 = sg0;
      Unit un2 = un1;
      if (u1 < n) sg1 = p.t.segs[un1.seg];
      if (u2 < n) un2 = p.t.units[u2];
      // the claim's result is first looked at when the unit indices rotate, at the loop's end
      unsigned int raw3 = 0xffffffffu;
      if (dyn && u2 < n) raw3 = atomicAdd(&p.ctr[0], 1u);
      const Unit &un = un0;
      const DevSeg &sg = sg0;
      const uint8_t *src_base = s_src[sg.src_rank] + sg.src_off;
      uint8_t *dst_base0 = s_dst[sg.dst_rank] + sg.dst_off;   // the first (often only) destination
      const bool long_run = sg.run_bytes >= T;
      const uint32_t tpr = long_run ? (uint32_t)((sg.run_bytes + T - 1) / T) : 1u;
      const uint32_t rpt = long_run ? 1u : (uint32_t)(T / sg.run_bytes);
      uint32_t run = long_run ? un.first_tile / tpr : un.first_tile * rpt;  // first run (row)
      uint32_t ch = long_run ? un.first_tile % tpr : 0u;                    // chunk in run
      for (uint32_t k = 0; k < un.n_tiles; ++k, ++it) {
        const uint32_t st = it % S, round = it / S;
        if (round > 0 && !mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) {
          ok = false;
          break;
        }
        if (s_abort) { ok = false; break; }
        uint32_t rows, row_bytes;
        uint64_t in_run;
        if (long_run) {
          in_run = (uint64_t)ch * T;
          const uint64_t left = sg.run_bytes - in_run;
          row_bytes = left < T ? (uint32_t)left : T;
          rows = 1;
        } else {
          in_run = 0;
          rows = sg.n_runs - run < rpt ? sg.n_runs - run : rpt;
          row_bytes = (uint32_t)sg.run_bytes;
        }
        TileInfo &ti = info[st];
        if (sg.n_dst == 1) {
          ti.dst_ptr[0] = (uint64_t)(dst_base0 + (uint64_t)run * sg.dst_pitch + in_run);
          ti.dst_pitch[0] = sg.dst_pitch;
        } else {
          for (uint32_t d = 0; d < sg.n_dst; ++d) {
            const Dst dd = p.t.dsts[sg.dst_first + d];
            ti.dst_ptr[d] = (uint64_t)(s_dst[dd.rank] + dd.off + (uint64_t)run * dd.pitch + in_run);
            ti.dst_pitch[d] = dd.pitch;
          }
        }
        ti.n_dst = sg.n_dst;
        ti.n_rows = rows;
        ti.row_bytes = row_bytes;
        if (p.pace_ns) {
          // bandwidth limit: a CTA's loads are spaced pace_ns per full tile apart (a short
          // tile earns a proportionally short gap); time not used is not saved up beyond
          // two tiles.  The sleep is at most one gap long.
          const unsigned long long burst = 2ull * p.pace_ns;
          unsigned long long now = globaltimer_ns();
          for (int spin = 0; now < t_next && spin < (1 << 16); ++spin) {
            __nanosleep(t_next - now < 1000 ? (unsigned)(t_next - now) : 1000u);
            now = globaltimer_ns();
          }
          if (t_next + burst < now) t_next = now - burst;
          t_next += (unsigned long long)p.pace_ns * (rows * row_bytes) / T;
        }
        const uint32_t bar = smem_u32(&full[st]);
        mbar_arrive_expect_tx(bar, rows * row_bytes);
        const uint8_t *sp = src_base + (uint64_t)run * sg.src_pitch + in_run;
        const uint32_t dp = smem_u32(data + (size_t)st * T);
        // rows that follow one another without a gap in the source are one load
        uint32_t n_ld = rows, ld_bytes = row_bytes;
        if (rows > 1 && sg.src_pitch == row_bytes) { n_ld = 1; ld_bytes = rows * row_bytes; }
        if (hint) {
          for (uint32_t r = 0; r < n_ld; ++r)
            bulk_load_hint(dp + r * ld_bytes, sp + (uint64_t)r * sg.src_pitch, ld_bytes, bar, pol);
        } else {
          for (uint32_t r = 0; r < n_ld; ++r)
            bulk_load(dp + r * ld_bytes, sp + (uint64_t)r * sg.src_pitch, ld_bytes, bar);
        }
        if (long_run) {
          if (++ch == tpr) { ch = 0; ++run; }
        } else {
          run += rows;
        }
      }
      un0 = un1;
      sg0 = sg1;
      un1 = un2;
      u = u1;
      u1 = u2;
      if (dyn) u2 = u2 < n ? claimed(raw3) : n;
      else u2 = (uint64_t)u2 + G < n ? u2 + G : n;
    }
    if (ok) {
      // end marker
      const uint32_t st = it % S, round = it / S;
      if (round == 0 || mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) {
        info[st].n_rows = 0;
        mbar_arrive(smem_u32(&full[st]));
      } else {
        ok = false;
      }
    }
    if (!ok) {
      // a wait expired: flag it, then let the loads already issued land before leaving
      s_abort = 1;
      atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
      const uint32_t back = it < S ? it : S;
      for (uint32_t j = 1; j <= back; ++j) {
        const uint32_t i2 = it - j;
        (void)mbar_wait(smem_u32(&full[i2 % S]), (i2 / S) & 1, kDrainLimitNs);
      }
    }
    if (dyn) {  // the last producer to finish leaves the counters at zero for the next launch
      __threadfence();
      if (atomicAdd(&p.ctr[1], 1u) == G - 1) {
        p.ctr[0] = 0;
        p.ctr[1] = 0;
        __threadfence();
      }
    }
  } else if (tid == 32) {
    // ---------------- consumer: issue stores, recycle stages ----------------
    // A stage is handed back one tile late: when the store of tile i has been issued,
    // the store of tile i-1 is waited for (reads of shared memory only) and its stage
    // released.  Releasing a stage right after its own store (a blocking wait per
    // tile) and several store-issuing threads were both measured slower.
    const uint64_t pol = policy_evict_first();
    const bool hint = (p.hints & 2u) != 0;
    for (uint32_t it = 0;; ++it) {
      const uint32_t st = it % S, round = it / S;
      if (!mbar_wait(smem_u32(&full[st]), round & 1, p.wait_ns, &s_abort)) {
        s_abort = 1;
        atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
        break;
      }
      const TileInfo &ti = info[st];
      const uint32_t rows = ti.n_rows, rb = ti.row_bytes;
      if (rows == 0) break;
      const uint32_t sp = smem_u32(data + (size_t)st * T);
      for (uint32_t d = 0; d < ti.n_dst; ++d) {
        uint8_t *dp = reinterpret_cast<uint8_t *>(ti.dst_ptr[d]);
        const uint64_t pitch = ti.dst_pitch[d];
        // rows that follow one another without a gap in the destination are one store
        uint32_t n_st = rows, sb = rb;
        if (rows > 1 && pitch == rb) { n_st = 1; sb = rows * rb; }
        if (hint) {
          for (uint32_t r = 0; r < n_st; ++r)
            bulk_store_hint(dp + (uint64_t)r * pitch, sp + r * sb, sb, pol);
        } else {
          for (uint32_t r = 0; r < n_st; ++r) bulk_store(dp + (uint64_t)r * pitch, sp + r * sb, sb);
        }
      }
      bulk_commit();
      if (it >= 1) {  // the store of the previous tile has finished reading its stage
        bulk_wait_read<1>();
        mbar_arrive(smem_u32(&empty[(it - 1) % S]));
      }
    }
    bulk_wait_read<0>();
  }
}

// ---- KV head re-split -------------------------------------------------------------------

struct KvParams {
  KvTables t;
  RankPtrs ptrs;
};

// Direct variant: thread q of a tile owns piece q of the LOGICAL block
// [token][global head][piece]; it reads the piece from the old rank that holds the
// head and writes it to the new rank that will.  Reads of a warp cover whole token
// rows of the old layout, writes whole head vectors of the new one.
// The CTA copies tiles first, first + stride, ... (a tile = one (layer, K|V, block pair)).
template <typename V>
__device__ __forceinline__ void kv_direct_tiles(const KvTables &t, const RankPtrs &ptrs, uint64_t first,
                                                uint64_t stride) {
  constexpr uint32_t W = sizeof(V);
  const uint32_t cpv = t.head_bytes / W;     // pieces per head vector
  const uint32_t row = t.hkv * cpv;          // pieces per logical token row
  const uint32_t total = t.block_tokens * row;
  const uint64_t blk_old = (uint64_t)t.block_tokens * t.hc * t.head_bytes;
  const uint64_t blk_new = (uint64_t)t.block_tokens * t.hn * t.head_bytes;
  const uint64_t n_tiles = (uint64_t)t.n_pairs * t.n_lk;
  for (uint64_t tile = first; tile < n_tiles; tile += stride) {
    const uint32_t lk = (uint32_t)(tile / t.n_pairs), pr = (uint32_t)(tile % t.n_pairs);
    const uint64_t base_old = ((uint64_t)lk * t.nb_old + t.pair_old[pr]) * blk_old;
    const uint64_t base_new = ((uint64_t)lk * t.nb_new + t.pair_new[pr]) * blk_new;
    for (uint32_t q0 = threadIdx.x; q0 < total; q0 += blockDim.x * 4) {
      V v[4];
      uint32_t tok[4], g[4], j[4];
      bool live[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t q = q0 + u * blockDim.x;
        live[u] = false;
        if (q < total) {
          tok[u] = q / row;
          const uint32_t rem = q - tok[u] * row;
          g[u] = rem / cpv;
          j[u] = rem - g[u] * cpv;
          live[u] = t.dst_only == 0xffffffffu || g[u] / t.hn == t.dst_only;
        }
        if (live[u]) {
          uint32_t ro = g[u] / t.hc, ho = g[u] - ro * t.hc;
          if (t.use_map) { ro = t.map_rank[g[u]]; ho = t.map_head[g[u]]; }
          v[u] = *reinterpret_cast<const V *>(
              ptrs.src[ro] + base_old + ((uint64_t)(tok[u] * t.hc + ho) * cpv + j[u]) * W);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (live[u]) {
          const uint32_t rn = g[u] / t.hn, hn = g[u] - rn * t.hn;
          *reinterpret_cast<V *>(ptrs.dst[rn] + base_new +
                                 ((uint64_t)(tok[u] * t.hn + hn) * cpv + j[u]) * W) = v[u];
        }
      }
    }
  }
}

template <typename V>
__global__ void __launch_bounds__(256) kv_direct_kernel(const __grid_constant__ KvParams p) {
  kv_direct_tiles<V>(p.t, p.ptrs, blockIdx.x, gridDim.x);
}

// Row-mapped variant of the direct kernel for the usual case that a CTA's 256 threads
// cover whole logical token rows (256 % pieces-per-row == 0): a thread then keeps the same
// (head, piece) for every token it touches, so its source / destination rank and in-block
// offsets are fixed for the whole kernel and a tile costs two base offsets, U loads and U
// stores.  The block ids of the next tile are fetched while the current one is in flight.
template <int U>
__device__ __forceinline__ void kv_rows_tiles(const KvTables &t, const RankPtrs &ptrs, uint64_t first,
                                              uint64_t stride) {
  const uint32_t cpv = t.head_bytes / 16, row = t.hkv * cpv, tpp = 256 / row;  // tokens per pass
  const uint32_t rem = threadIdx.x % row, tok0 = threadIdx.x / row;
  const uint32_t g = rem / cpv, j = rem - g * cpv;
  uint32_t ro = g / t.hc, ho = g - ro * t.hc;
  if (t.use_map) { ro = t.map_rank[g]; ho = t.map_head[g]; }
  const uint32_t rn = g / t.hn, hn = g - rn * t.hn;
  if (t.dst_only != 0xffffffffu && rn != t.dst_only) return;  // another rank writes that block
  const uint8_t *sp = ptrs.src[ro] + ((uint64_t)(tok0 * t.hc + ho) * cpv + j) * 16;
  uint8_t *dp = ptrs.dst[rn] + ((uint64_t)(tok0 * t.hn + hn) * cpv + j) * 16;
  const uint64_t s_step = (uint64_t)tpp * t.hc * t.head_bytes, d_step = (uint64_t)tpp * t.hn * t.head_bytes;
  const uint64_t blk_old = (uint64_t)t.block_tokens * t.hc * t.head_bytes;
  const uint64_t blk_new = (uint64_t)t.block_tokens * t.hn * t.head_bytes;
  const uint64_t n_tiles = (uint64_t)t.n_pairs * t.n_lk;
  uint64_t tile = first;
  if (tile >= n_tiles) return;
  uint32_t lk = (uint32_t)(tile / t.n_pairs), pr = (uint32_t)(tile - (uint64_t)lk * t.n_pairs);
  uint32_t po = t.pair_old[pr], pn = t.pair_new[pr];
  for (;;) {
    const uint64_t tile2 = tile + stride;
    uint32_t lk2 = lk, po2 = po, pn2 = pn;
    if (tile2 < n_tiles) {
      lk2 = (uint32_t)(tile2 / t.n_pairs);
      const uint32_t pr2 = (uint32_t)(tile2 - (uint64_t)lk2 * t.n_pairs);
      po2 = t.pair_old[pr2];
      pn2 = t.pair_new[pr2];
    }
    const uint8_t *s = sp + ((uint64_t)lk * t.nb_old + po) * blk_old;
    uint8_t *d = dp + ((uint64_t)lk * t.nb_new + pn) * blk_new;
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (tok0 + u * tpp < t.block_tokens) v[u] = *reinterpret_cast<const uint4 *>(s + u * s_step);
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (tok0 + u * tpp < t.block_tokens) *reinterpret_cast<uint4 *>(d + u * d_step) = v[u];
    if (tile2 >= n_tiles) break;
    tile = tile2; lk = lk2; po = po2; pn = pn2;
  }
}

template <int U>
__global__ void __launch_bounds__(256) kv_rows_kernel(const __grid_constant__ KvParams p) {
  kv_rows_tiles<U>(p.t, p.ptrs, blockIdx.x, gridDim.x);
}

// Passes the row-mapped copy needs for a block (0: the shape does not fit it).
__host__ __device__ inline uint32_t kv_rows_passes(const KvTables &t) {
  if (t.head_bytes % 16) return 0;
  const uint32_t row = t.hkv * (t.head_bytes / 16);
  if (row == 0 || row > 256 || 256 % row) return 0;
  return (t.block_tokens + 256 / row - 1) / (256 / row);
}

// ---- vector path ------------------------------------------------------------------------

struct VecParams {
  SegTables t;
  uint32_t tile_bytes;
  RankPtrs ptrs;
};

// The vector kernel with the tiles of a KV head re-split appended to its work: CTAs
// [0, vec_ctas) walk the segment units, the others the KV tiles.  One launch then covers
// a whole TP-changing step whose phases are too small for a launch each.
struct VecKvParams {
  SegTables t;
  uint32_t tile_bytes;
  uint32_t vec_ctas;     // CTAs that take segment units
  uint32_t kv_passes;    // row-mapped copy: passes per block (1, 2, 4, 8); 0: the direct copy
  RankPtrs ptrs;         // segment arenas
  KvTables kv;
  RankPtrs kv_ptrs;      // KV arenas
};

// One warp copies one tile to one destination: `rows` rows of cpr pieces, a pitch apart
// on either side.  Lanes keep a fixed column (or, for rows shorter than a warp pass, a
// fixed sub-row and column), so the steady state has no division; four loads are in
// flight per lane before the stores.
template <typename V>
__device__ __forceinline__ void warp_copy_tile(const uint8_t *sp, uint64_t src_pitch, uint8_t *dp,
                                               uint64_t dst_pitch, uint32_t rows, uint32_t cpr,
                                               uint32_t lane) {
  if (cpr >= 32) {
#pragma unroll 1
    for (uint32_t r = 0; r < rows; ++r) {
      const V *srow = reinterpret_cast<const V *>(sp + (uint64_t)r * src_pitch);
      V *drow = reinterpret_cast<V *>(dp + (uint64_t)r * dst_pitch);
#pragma unroll 1
      for (uint32_t c0 = lane; c0 < cpr; c0 += 32 * 4) {
        V v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 32 * u < cpr) v[u] = srow[c0 + 32 * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 32 * u < cpr) drow[c0 + 32 * u] = v[u];
      }
    }
  } else {
    const uint32_t rpp = 32 / cpr;  // rows per warp pass
    const uint32_t sub = lane / cpr, c = lane - sub * cpr;
    if (sub >= rpp) return;
#pragma unroll 1
    for (uint32_t r0 = sub; r0 < rows; r0 += rpp * 4) {
      V v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (r0 + rpp * u < rows)
          v[u] = reinterpret_cast<const V *>(sp + (uint64_t)(r0 + rpp * u) * src_pitch)[c];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (r0 + rpp * u < rows)
          reinterpret_cast<V *>(dp + (uint64_t)(r0 + rpp * u) * dst_pitch)[c] = v[u];
    }
  }
}

// A CTA takes one unit at a time (its segment is parked in shared memory), a warp one tile.
// The CTA walks units first, first + stride, ...
__device__ __forceinline__ void vec_copy_units(const SegTables &t, const RankPtrs &ptrs, uint32_t T,
                                               uint32_t first, uint32_t stride) {
  __shared__ DevSeg s_sg;
  __shared__ Unit s_un;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (uint64_t u64 = first; u64 < t.n_units; u64 += stride) {
    const uint32_t u = (uint32_t)u64;
    __syncthreads();  // everyone is done with the previous unit's segment
    if (threadIdx.x == 0) s_un = t.units[u];
    if (threadIdx.x < 4) {
      const uint32_t seg = t.units[u].seg;
      reinterpret_cast<uint4 *>(&s_sg)[threadIdx.x] =
          reinterpret_cast<const uint4 *>(&t.segs[seg])[threadIdx.x];
    }
    __syncthreads();
    const uint64_t run_bytes = s_sg.run_bytes;
    const bool long_run = run_bytes >= T;
    const uint32_t tpr = long_run ? (uint32_t)((run_bytes + T - 1) / T) : 1u;
    const uint32_t rpt = long_run ? 1u : (uint32_t)(T / run_bytes);
    for (uint32_t k = warp; k < s_un.n_tiles; k += n_warps) {
      const uint32_t tile = s_un.first_tile + k;
      uint32_t run, rows, row_bytes;
      uint64_t in_run;
      if (long_run) {
        run = tile / tpr;
        in_run = (uint64_t)(tile % tpr) * T;
        const uint64_t left = run_bytes - in_run;
        row_bytes = left < T ? (uint32_t)left : T;
        rows = 1;
      } else {
        run = tile * rpt;
        in_run = 0;
        rows = s_sg.n_runs - run < rpt ? s_sg.n_runs - run : rpt;
        row_bytes = (uint32_t)run_bytes;
      }
      const uint64_t src_pitch = s_sg.src_pitch;
      const uint8_t *sp = ptrs.src[s_sg.src_rank] + s_sg.src_off + (uint64_t)run * src_pitch + in_run;
      const uint32_t n_dst = s_sg.n_dst, align = s_sg.align;
      for (uint32_t d = 0; d < n_dst; ++d) {
        uint64_t d_off = s_sg.dst_off, d_pitch = s_sg.dst_pitch;
        uint32_t d_rank = s_sg.dst_rank;
        if (n_dst > 1) {
          const Dst dd = t.dsts[s_sg.dst_first + d];
          d_off = dd.off; d_pitch = dd.pitch; d_rank = dd.rank;
        }
        uint8_t *dp = ptrs.dst[d_rank] + d_off + (uint64_t)run * d_pitch + in_run;
        switch (align) {
          case 16: warp_copy_tile<uint4>(sp, src_pitch, dp, d_pitch, rows, row_bytes / 16, lane); break;
          case 8: warp_copy_tile<uint2>(sp, src_pitch, dp, d_pitch, rows, row_bytes / 8, lane); break;
          case 4: warp_copy_tile<uint32_t>(sp, src_pitch, dp, d_pitch, rows, row_bytes / 4, lane); break;
          case 2: warp_copy_tile<uint16_t>(sp, src_pitch, dp, d_pitch, rows, row_bytes / 2, lane); break;
          default: warp_copy_tile<uint8_t>(sp, src_pitch, dp, d_pitch, rows, row_bytes, lane); break;
        }
      }
    }
  }
}

__global__ void __launch_bounds__(256, 4) vec_copy_kernel(const __grid_constant__ VecParams p) {
  vec_copy_units(p.t, p.ptrs, p.tile_bytes, blockIdx.x, gridDim.x);
}

__global__ void __launch_bounds__(256, 4) vec_kv_kernel(const __grid_constant__ VecKvParams p) {
  if (blockIdx.x < p.vec_ctas) {
    vec_copy_units(p.t, p.ptrs, p.tile_bytes, blockIdx.x, p.vec_ctas);
    return;
  }
  const uint64_t first = blockIdx.x - p.vec_ctas, stride = gridDim.x - p.vec_ctas;
  switch (p.kv_passes) {
    case 1: kv_rows_tiles<1>(p.kv, p.kv_ptrs, first, stride); break;
    case 2: kv_rows_tiles<2>(p.kv, p.kv_ptrs, first, stride); break;
    case 4: kv_rows_tiles<4>(p.kv, p.kv_ptrs, first, stride); break;
    case 8: kv_rows_tiles<8>(p.kv, p.kv_ptrs, first, stride); break;
    default: kv_direct_tiles<uint4>(p.kv, p.kv_ptrs, first, stride); break;
  }
}

// Staged variant: the fused gather-transpose through shared memory, with the copy engine on
// both sides.  One producer thread brings the c contiguous pieces of a logical block (one
// per old rank, each [token][local head][head_dim]) into a stage of an input ring with
// cp.async.bulk; 256 consumer threads transpose the stage inside shared memory into an
// output stage laid out as the d new blocks ([token][new local head][head_dim] each); one
// of them then issues one cp.async.bulk store per new rank.  No global load or store goes
// through the load/store units.  The input -> output piece mapping is the same for every
// tile, so it is tabulated once per CTA (no division in the steady state).
constexpr uint32_t kKvConsumers = 256;
constexpr uint32_t kKvOutStages = 2;
constexpr uint32_t kKvStagedCtasPerSm = 2;  // the per-tile chain of waits and barriers is long: overlap two CTAs

struct KvStagedParams {
  KvTables t;
  uint32_t stages, tile_bytes, n_pieces, chunk_bytes;  // chunk = one old rank's share of a block
  unsigned long long wait_ns;
  int *status;
  RankPtrs ptrs;
};

__device__ __forceinline__ void consumers_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kKvConsumers) : "memory");
}

__global__ void __launch_bounds__(kKvConsumers + 32, kKvStagedCtasPerSm)
kv_staged_kernel(const __grid_constant__ KvStagedParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const KvTables &t = p.t;
  const uint32_t S = p.stages, T = p.tile_bytes;
  uint8_t *data = smem;                                   // input ring: S stages, old layout
  uint8_t *out = smem + (size_t)S * T;                    // output ring: kKvOutStages, new layout
  uint32_t *table = reinterpret_cast<uint32_t *>(out + (size_t)kKvOutStages * T);
  uint64_t *base_new_of = reinterpret_cast<uint64_t *>(table + 2 * ((p.n_pieces + 1) / 2));  // per stage
  uint64_t *full = base_new_of + S;
  uint64_t *empty = full + S;
  __shared__ const uint8_t *s_src[EMOE_MAX_RANKS];
  __shared__ uint8_t *s_dst[EMOE_MAX_RANKS];
  __shared__ volatile int s_abort;
  __shared__ volatile int s_go;  // consumer 0 -> all consumers: 1 tile ready, 0 leave
  constexpr uint64_t kEnd = ~0ull;

  const uint32_t tid = threadIdx.x;
  if (tid < EMOE_MAX_RANKS) {
    s_src[tid] = p.ptrs.src[tid];
    s_dst[tid] = p.ptrs.dst[tid];
  }
  // input-stage offset of every 16-byte piece of the output stage (new-layout order)
  {
    const uint32_t cpv = t.head_bytes / 16, row_new = t.hn * cpv, ppr = t.block_tokens * row_new;
    for (uint32_t q = tid; q < p.n_pieces; q += blockDim.x) {
      const uint32_t rn = q / ppr, r = q - rn * ppr;
      const uint32_t tok = r / row_new, rem = r - tok * row_new;
      const uint32_t hl = rem / cpv, j = rem - hl * cpv;
      const uint32_t g = rn * t.hn + hl, ro = g / t.hc, ho = g - ro * t.hc;
      table[q] = ro * p.chunk_bytes + ((tok * t.hc + ho) * cpv + j) * 16;
    }
  }
  if (tid == 0) {
    s_abort = 0;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();

  const uint64_t blk_old = (uint64_t)p.chunk_bytes;
  const uint32_t blk_new = t.block_tokens * t.hn * t.head_bytes;
  const uint64_t n_tiles = (uint64_t)t.n_pairs * t.n_lk;
  const uint32_t c = t.hkv / t.hc, d = t.hkv / t.hn;

  if (tid == kKvConsumers) {
    // ---------------- producer ----------------
    uint32_t it = 0;
    bool ok = true;
    uint64_t tile = blockIdx.x;   // < n_tiles: the grid never exceeds the tile count
    uint32_t lk = (uint32_t)(tile / t.n_pairs), pr = (uint32_t)(tile % t.n_pairs);
    uint32_t po = t.pair_old[pr], pn = t.pair_new[pr];
    for (; tile < n_tiles; tile += gridDim.x, ++it) {
      // ids of the next tile are fetched now and used one iteration later
      const uint64_t tile2 = tile + gridDim.x;
      uint32_t lk2 = lk, pr2 = pr, po2 = po, pn2 = pn;
      if (tile2 < n_tiles) {
        lk2 = (uint32_t)(tile2 / t.n_pairs);
        pr2 = (uint32_t)(tile2 - (uint64_t)lk2 * t.n_pairs);
        po2 = t.pair_old[pr2];
        pn2 = t.pair_new[pr2];
      }
      const uint32_t st = it % S, round = it / S;
      if (round > 0 && !mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) { ok = false; break; }
      if (s_abort) { ok = false; break; }
      base_new_of[st] = ((uint64_t)lk * t.nb_new + pn) * blk_new;
      const uint64_t base_old = ((uint64_t)lk * t.nb_old + po) * blk_old;
      const uint32_t bar = smem_u32(&full[st]);
      mbar_arrive_expect_tx(bar, T);
      const uint32_t dp = smem_u32(data + (size_t)st * T);
      for (uint32_t ro = 0; ro < c; ++ro)
        bulk_load(dp + ro * p.chunk_bytes, s_src[ro] + base_old, p.chunk_bytes, bar);
      lk = lk2; pr = pr2; po = po2; pn = pn2;
    }
    if (ok) {  // end marker
      const uint32_t st = it % S, round = it / S;
      if (round == 0 || mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) {
        base_new_of[st] = kEnd;
        mbar_arrive(smem_u32(&full[st]));
      } else {
        ok = false;
      }
    }
    if (!ok) {
      // a wait expired: flag it, then let the loads already issued land before leaving
      s_abort = 1;
      atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
      const uint32_t back = it < S ? it : S;
      for (uint32_t j = 1; j <= back; ++j) {
        const uint32_t i2 = it - j;
        (void)mbar_wait(smem_u32(&full[i2 % S]), (i2 / S) & 1, kDrainLimitNs);
      }
    }
  } else if (tid < kKvConsumers) {
    // ---------------- consumers ----------------
    // Consumer 0 does every wait (bounded) and tells the others through s_go, so that all
    // 256 leave the loop in the same iteration and no named barrier is left short.
    const uint32_t n = p.n_pieces;
    for (uint32_t it = 0;; ++it) {
      const uint32_t st = it % S, round = it / S, os = it % kKvOutStages;
      if (tid == 0) {
        int go = 1;
        if (!mbar_wait(smem_u32(&full[st]), round & 1, p.wait_ns, &s_abort)) {
          s_abort = 1;
          atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
          go = 0;
        } else if (base_new_of[st] == kEnd) {
          go = 0;
        }
        // the stores issued kKvOutStages tiles ago have finished reading this output stage
        bulk_wait_read<kKvOutStages - 1>();
        s_go = go;
      }
      consumers_sync();
      if (!s_go) break;
      const uint8_t *stage = data + (size_t)st * T;
      uint8_t *ostage = out + (size_t)os * T;
      for (uint32_t q0 = tid; q0 < n; q0 += kKvConsumers * 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t q = q0 + u * kKvConsumers;
          if (q < n) v[u] = *reinterpret_cast<const uint4 *>(stage + table[q]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t q = q0 + u * kKvConsumers;
          if (q < n) *reinterpret_cast<uint4 *>(ostage + (size_t)q * 16) = v[u];
        }
      }
      fence_proxy_async_smem();   // the transposed stage becomes visible to the copy engine
      consumers_sync();           // ... and everyone is done with the input stage
      if (tid == 0) {
        const uint64_t base_new = base_new_of[st];
        const uint32_t sp = smem_u32(ostage);
        for (uint32_t rn = 0; rn < d; ++rn)
          bulk_store(s_dst[rn] + base_new, sp + rn * blk_new, blk_new);
        bulk_commit();
        mbar_arrive(smem_u32(&empty[st]));
      }
    }
    if (tid == 0) bulk_wait_read<0>();
  }
}

// Tensor-map variant: the copy engine does the gather-transpose.  Every arena is
// described to TMA as a 3-D tensor [token rows][local heads][head bytes]; a box of
// (block_tokens x g heads x head bytes), g = gcd(heads per old rank, heads per new
// rank), is contiguous in neither layout but is one tiled load from the old arena and
// one tiled store into the new one.  One thread issues the loads of a block pair into a
// stage of the ring, one thread the stores: no data passes through registers.
constexpr uint32_t kKvTmaMaxBoxes = 64;

struct KvTmaParams {
  KvTables t;
  uint32_t stages, tile_bytes, box_bytes, n_box, g;
  unsigned long long wait_ns;
  int *status;
  CUtensorMap src[kKvTmaMaxRanks], dst[kKvTmaMaxRanks];
};

__global__ void __launch_bounds__(64, 1) kv_tma_kernel(const __grid_constant__ KvTmaParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const KvTables &t = p.t;
  const uint32_t S = p.stages, T = p.tile_bytes;
  uint8_t *data = smem;
  int32_t *tok_new_of = reinterpret_cast<int32_t *>(smem + (size_t)S * T);  // per stage, -1 = end
  uint64_t *full = reinterpret_cast<uint64_t *>(tok_new_of + 2 * ((S + 1) / 2));
  uint64_t *empty = full + S;
  // per box: old rank, head offset inside it, new rank, head offset inside it
  __shared__ uint8_t b_ro[kKvTmaMaxBoxes], b_rn[kKvTmaMaxBoxes];
  __shared__ uint16_t b_ho[kKvTmaMaxBoxes], b_hn[kKvTmaMaxBoxes];
  __shared__ volatile int s_abort;

  const uint32_t tid = threadIdx.x;
  if (tid < p.n_box) {
    const uint32_t h = tid * p.g, ro = h / t.hc, rn = h / t.hn;
    b_ro[tid] = (uint8_t)ro;
    b_rn[tid] = (uint8_t)rn;
    b_ho[tid] = (uint16_t)(h - ro * t.hc);
    b_hn[tid] = (uint16_t)(h - rn * t.hn);
  }
  if (tid == 0) {
    s_abort = 0;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();

  const uint64_t n_tiles = (uint64_t)t.n_pairs * t.n_lk;
  if (tid == 0) {
    // ---------------- producer ----------------
    uint32_t it = 0;
    bool ok = true;
    uint64_t tile = blockIdx.x;   // < n_tiles: the grid never exceeds the tile count
    uint32_t lk = (uint32_t)(tile / t.n_pairs), pr = (uint32_t)(tile % t.n_pairs);
    uint32_t po = t.pair_old[pr], pn = t.pair_new[pr];
    for (; tile < n_tiles; tile += gridDim.x, ++it) {
      // ids of the next tile are fetched now and used one iteration later
      const uint64_t tile2 = tile + gridDim.x;
      uint32_t lk2 = lk, pr2 = pr, po2 = po, pn2 = pn;
      if (tile2 < n_tiles) {
        lk2 = (uint32_t)(tile2 / t.n_pairs);
        pr2 = (uint32_t)(tile2 - (uint64_t)lk2 * t.n_pairs);
        po2 = t.pair_old[pr2];
        pn2 = t.pair_new[pr2];
      }
      const uint32_t st = it % S, round = it / S;
      if (round > 0 && !mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) { ok = false; break; }
      if (s_abort) { ok = false; break; }
      // first token row of the block in the old / new arena tensors (< 2^31, checked on the host)
      const int32_t tok_old = (int32_t)(((uint64_t)lk * t.nb_old + po) * t.block_tokens);
      tok_new_of[st] = (int32_t)(((uint64_t)lk * t.nb_new + pn) * t.block_tokens);
      const uint32_t bar = smem_u32(&full[st]);
      mbar_arrive_expect_tx(bar, T);
      const uint32_t dp = smem_u32(data + (size_t)st * T);
      for (uint32_t k = 0; k < p.n_box; ++k)
        tma_load_3d(dp + k * p.box_bytes, &p.src[b_ro[k]], 0, (int32_t)b_ho[k], tok_old, bar);
      lk = lk2; pr = pr2; po = po2; pn = pn2;
    }
    if (ok) {  // end marker
      const uint32_t st = it % S, round = it / S;
      if (round == 0 || mbar_wait(smem_u32(&empty[st]), (round - 1) & 1, p.wait_ns, &s_abort)) {
        tok_new_of[st] = -1;
        mbar_arrive(smem_u32(&full[st]));
      } else {
        ok = false;
      }
    }
    if (!ok) {
      // a wait expired: flag it, then let the loads already issued land before leaving
      s_abort = 1;
      atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
      const uint32_t back = it < S ? it : S;
      for (uint32_t j = 1; j <= back; ++j) {
        const uint32_t i2 = it - j;
        (void)mbar_wait(smem_u32(&full[i2 % S]), (i2 / S) & 1, kDrainLimitNs);
      }
    }
  } else if (tid == 32) {
    // ---------------- consumer ----------------
    for (uint32_t it = 0;; ++it) {
      const uint32_t st = it % S, round = it / S;
      if (!mbar_wait(smem_u32(&full[st]), round & 1, p.wait_ns, &s_abort)) {
        s_abort = 1;
        atomicExch(p.status, (int)EMOE_ERR_DEVICE_TIMEOUT);
        break;
      }
      const int32_t tok_new = tok_new_of[st];
      if (tok_new < 0) break;
      const uint32_t sp = smem_u32(data + (size_t)st * T);
      for (uint32_t k = 0; k < p.n_box; ++k)
        tma_store_3d(&p.dst[b_rn[k]], 0, (int32_t)b_hn[k], tok_new, sp + k * p.box_bytes);
      bulk_commit();
      if (it >= 1) {  // the stores of the previous tile have finished reading its stage
        bulk_wait_read<1>();
        mbar_arrive(smem_u32(&empty[(it - 1) % S]));
      }
    }
    bulk_wait_read<0>();
  }
}

}  // namespace

// ---- launchers --------------------------------------------------------------------------

size_t bulk_smem_bytes(uint32_t tile_bytes, uint32_t stages) {
  return (size_t)stages * tile_bytes + stages * (sizeof(TileInfo) + 2 * sizeof(uint64_t));
}

size_t bulk_smem_limit() { return kBulkSmemLimit; }

// Dynamic shared memory opt-in of the ring kernels.  The attribute belongs to the device
// that is current when it is set, so this runs once per device ordinal.
cudaError_t kernels_init() {
  static std::mutex mu;
  static bool done[kMaxDevices] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(bulk_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)kBulkSmemLimit);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kv_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kv_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  done[dev] = true;
  return cudaSuccess;
}

cudaError_t launch_bulk_copy(const SegTables &t, const RankPtrs &ptrs, const BulkConfig &c,
                             uint32_t grid, int *status, unsigned int *ctr, cudaStream_t stream) {
  if (t.n_units == 0) return cudaSuccess;
  if (c.stages < 2 || c.stages > kMaxStages || c.tile_bytes % 128 != 0) return cudaErrorInvalidValue;
  const size_t smem = bulk_smem_bytes(c.tile_bytes, c.stages);
  if (smem > kBulkSmemLimit) return cudaErrorInvalidValue;
  BulkParams p{t, c.tile_bytes, c.stages, c.hints, c.pace_ns, c.wait_ns, status, ctr, ptrs};
  if (grid > t.n_units) grid = t.n_units;
  bulk_copy_kernel<<<grid, 64, smem, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_vec_copy(const SegTables &t, const RankPtrs &ptrs, uint32_t tile_bytes,
                            uint32_t grid, cudaStream_t stream) {
  if (t.n_units == 0) return cudaSuccess;
  VecParams p{t, tile_bytes, ptrs};
  if (grid > t.n_units) grid = t.n_units;
  vec_copy_kernel<<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

bool vec_kv_supported(const KvTables &kv) { return kv.head_bytes % 16 == 0; }

cudaError_t launch_vec_kv_copy(const SegTables &t, const RankPtrs &ptrs, uint32_t tile_bytes,
                               const KvTables &kv, const RankPtrs &kv_ptrs, uint32_t grid,
                               bool unbounded, cudaStream_t stream) {
  const uint64_t n_tiles = (uint64_t)kv.n_pairs * kv.n_lk;
  if (n_tiles == 0) return launch_vec_copy(t, ptrs, tile_bytes, unbounded ? 0xffffffffu : grid, stream);
  VecKvParams p{};
  p.t = t;
  p.tile_bytes = tile_bytes;
  p.ptrs = ptrs;
  p.kv = kv;
  p.kv_ptrs = kv_ptrs;
  const uint32_t passes = kv_rows_passes(kv);
  p.kv_passes = passes == 1 ? 1 : passes == 2 ? 2 : passes >= 3 && passes <= 4 ? 4 :
                passes >= 5 && passes <= 8 ? 8 : 0;
  // no budget: one CTA per segment unit and one per KV tile (the hardware scheduler balances
  // them); with a budget the CTAs are split in proportion to the two kinds of work
  uint64_t vec_ctas, kv_ctas;
  if (unbounded) {
    vec_ctas = t.n_units;
    kv_ctas = n_tiles;
  } else {
    if (grid < 2) grid = 2;
    vec_ctas = t.n_units == 0 ? 0 : (uint64_t)grid * t.n_units / (t.n_units + n_tiles);
    if (t.n_units && vec_ctas == 0) vec_ctas = 1;
    if (vec_ctas > t.n_units) vec_ctas = t.n_units;
    kv_ctas = grid - vec_ctas;
    if (kv_ctas > n_tiles) kv_ctas = n_tiles;
  }
  if (vec_ctas + kv_ctas > 0x7fffffffull) kv_ctas = 0x7fffffffull - vec_ctas;
  p.vec_ctas = (uint32_t)vec_ctas;
  vec_kv_kernel<<<(uint32_t)(vec_ctas + kv_ctas), 256, 0, stream>>>(p);
  return cudaGetLastError();
}

namespace {
size_t kv_staged_smem(uint32_t tile_bytes, uint32_t stages) {
  const size_t pieces = tile_bytes / 16;
  return (size_t)(stages + kKvOutStages) * tile_bytes + 2 * ((pieces + 1) / 2) * sizeof(uint32_t) +
         (size_t)stages * 3 * sizeof(uint64_t);
}
}  // namespace

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                   const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link against libcuda).
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      p = nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

uint32_t gcd_u32(uint32_t a, uint32_t b) {
  while (b) { const uint32_t r = a % b; a = b; b = r; }
  return a;
}

size_t kv_tma_smem(uint32_t tile_bytes, uint32_t stages) {
  return (size_t)stages * tile_bytes + (size_t)(2 * ((stages + 1) / 2)) * sizeof(int32_t) +
         (size_t)stages * 2 * sizeof(uint64_t);
}

// One arena as a 3-D tensor [token rows][heads][head bytes in `es`-byte elements].
bool encode_arena(CUtensorMap *m, const void *base, uint32_t head_bytes, uint32_t heads,
                  uint64_t token_rows, uint32_t box_heads, uint32_t box_tokens) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const uint32_t es = head_bytes % 4 == 0 ? 4 : 1;
  const cuuint64_t dims[3] = {head_bytes / es, heads, token_rows};
  const cuuint64_t strides[2] = {head_bytes, (cuuint64_t)heads * head_bytes};
  const cuuint32_t box[3] = {head_bytes / es, box_heads, box_tokens};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, es == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
             const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool kv_tma_supported(const KvTables &t, uint32_t *stages_out) {
  const uint32_t c = t.hkv / t.hc, d = t.hkv / t.hn, g = gcd_u32(t.hc, t.hn);
  const uint32_t hb = t.head_bytes;
  const uint64_t tile = (uint64_t)t.block_tokens * t.hkv * hb;
  const uint64_t box = (uint64_t)t.block_tokens * g * hb;
  const uint64_t rows_old = (uint64_t)t.n_lk * t.nb_old * t.block_tokens;
  const uint64_t rows_new = (uint64_t)t.n_lk * t.nb_new * t.block_tokens;
  if (t.use_map || t.dst_only != 0xffffffffu || hb % 16 || c > kKvTmaMaxRanks || d > kKvTmaMaxRanks)
    return false;
  if ((hb % 4 == 0 ? hb / 4 : hb) > 256 || g > 256 || t.block_tokens > 256) return false;  // box extents
  if (box % 128 || t.hkv / g > kKvTmaMaxBoxes || tile > 96 * 1024) return false;
  if (rows_old >= (1ull << 31) || rows_new >= (1ull << 31)) return false;             // int32 coordinates
  uint32_t stages = (uint32_t)((192 * 1024) / tile);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2 || !encode_tiled_fn()) return false;
  if (stages_out) *stages_out = stages;
  return true;
}

bool kv_staged_supported(const KvTables &t, uint32_t *stages_out) {
  const uint64_t tile = (uint64_t)t.block_tokens * t.hkv * t.head_bytes;
  const uint64_t blk_new = (uint64_t)t.block_tokens * t.hn * t.head_bytes;
  if (t.use_map || t.dst_only != 0xffffffffu) return false;  // only the default kernels do these
  if (t.head_bytes % 16 || tile > 24 * 1024 || blk_new >= (1u << 24) || t.hkv / t.hn > 255) return false;
  uint32_t stages = (uint32_t)((100 * 1024) / tile);            // two CTAs per SM
  stages = stages > kKvOutStages ? stages - kKvOutStages : 0;   // the output ring takes two
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  if (stages_out) *stages_out = stages;
  return true;
}

cudaError_t launch_kv_copy(const KvTables &t, const RankPtrs &ptrs, int mode, uint32_t grid,
                           bool unbounded, int *status, unsigned long long wait_ns,
                           cudaStream_t stream) {
  const uint64_t n_tiles = (uint64_t)t.n_pairs * t.n_lk;
  if (n_tiles == 0) return cudaSuccess;
  KvParams p{t, ptrs};
  const uint32_t hb = t.head_bytes;
  uint32_t stages = 0;
  if (mode == 3 && status && kv_tma_supported(t, &stages)) {
    const uint32_t c = t.hkv / t.hc, d = t.hkv / t.hn, g = gcd_u32(t.hc, t.hn);
    KvTmaParams tp{};
    tp.t = t;
    tp.stages = stages;
    tp.tile_bytes = t.block_tokens * t.hkv * hb;
    tp.box_bytes = t.block_tokens * g * hb;
    tp.n_box = t.hkv / g;
    tp.g = g;
    tp.wait_ns = wait_ns;
    tp.status = status;
    bool ok = true;
    for (uint32_t r = 0; ok && r < c; ++r)
      ok = encode_arena(&tp.src[r], ptrs.src[r], hb, t.hc, (uint64_t)t.n_lk * t.nb_old * t.block_tokens,
                        g, t.block_tokens);
    for (uint32_t r = 0; ok && r < d; ++r)
      ok = encode_arena(&tp.dst[r], ptrs.dst[r], hb, t.hn, (uint64_t)t.n_lk * t.nb_new * t.block_tokens,
                        g, t.block_tokens);
    if (ok) {
      if (grid > n_tiles) grid = (uint32_t)n_tiles;
      kv_tma_kernel<<<grid, 64, kv_tma_smem(tp.tile_bytes, stages), stream>>>(tp);
      return cudaGetLastError();
    }
    // a tensor map could not be encoded: fall through to the direct kernel
  }
  if (mode == 2 && status && kv_staged_supported(t, &stages)) {
    const uint32_t tile = t.block_tokens * t.hkv * hb;
    KvStagedParams sp{t, stages, tile, tile / 16, t.block_tokens * t.hc * hb, wait_ns, status, ptrs};
    // two CTAs per budgeted SM; with no budget, 1.5 per SM measured best (6.6 TB/s on the
    // large-expert-count shape against 6.0 with 2 and 5.6 with 1)
    grid = unbounded ? grid * 3 / 2 : grid * kKvStagedCtasPerSm;
    if (grid > n_tiles) grid = (uint32_t)n_tiles;
    kv_staged_kernel<<<grid, kKvConsumers + 32, kv_staged_smem(tile, stages), stream>>>(sp);
    return cudaGetLastError();
  }
  // Direct kernels: with no CTA budget, one CTA per tile - the hardware block scheduler
  // balances better than any grid-stride loop (measured: 5.9 -> 6.6 TB/s); with a budget,
  // eight small CTAs per budgeted SM walk the tiles.
  const uint64_t want = unbounded ? n_tiles : (uint64_t)grid * 8;
  grid = (uint32_t)(want < n_tiles ? want : n_tiles);
  if (n_tiles > 0x7fffffffull && unbounded) grid = 0x7fffffffu;
  if (mode != 4) {
    // whole token rows per CTA pass, and few enough passes: the row-mapped kernel
    const uint32_t passes = kv_rows_passes(t);
    if (passes == 1) { kv_rows_kernel<1><<<grid, 256, 0, stream>>>(p); return cudaGetLastError(); }
    if (passes == 2) { kv_rows_kernel<2><<<grid, 256, 0, stream>>>(p); return cudaGetLastError(); }
    if (passes >= 3 && passes <= 4) { kv_rows_kernel<4><<<grid, 256, 0, stream>>>(p); return cudaGetLastError(); }
    if (passes >= 5 && passes <= 8) { kv_rows_kernel<8><<<grid, 256, 0, stream>>>(p); return cudaGetLastError(); }
  }
  if (hb % 16 == 0) kv_direct_kernel<uint4><<<grid, 256, 0, stream>>>(p);
  else if (hb % 8 == 0) kv_direct_kernel<uint2><<<grid, 256, 0, stream>>>(p);
  else if (hb % 4 == 0) kv_direct_kernel<uint32_t><<<grid, 256, 0, stream>>>(p);
  else if (hb % 2 == 0) kv_direct_kernel<uint16_t><<<grid, 256, 0, stream>>>(p);
  else kv_direct_kernel<uint8_t><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

// ---- unit tables expanded on the device ---------------------------------------------------
//
// A phase whose bulk segments all have the same number of runs, each run at least a tile
// long, has a regular unit table: run-major, and inside a run segment after segment.  The
// host then only sends, per segment, where its units start inside a run; one thread per
// (segment, run) writes that segment's units of that run.

namespace {
__global__ void gen_units_kernel(const DevSeg *segs, const uint32_t *seg_idx, const uint32_t *seg_pre,
                                 uint32_t n_segs, uint32_t n_runs, uint32_t group, uint32_t units_per_group,
                                 uint32_t tile_bytes, uint32_t unit_tiles, uint32_t seg_offset,
                                 Unit *out) {
  const uint32_t n_groups = (n_runs + group - 1) / group;
  const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (uint64_t)n_segs * n_groups) return;
  const uint32_t k = (uint32_t)(i % n_segs), grp = (uint32_t)(i / n_segs);
  const uint32_t seg = seg_idx[k] + seg_offset;
  const uint64_t run_bytes = segs[seg].run_bytes;
  const uint32_t tpr = (uint32_t)((run_bytes + tile_bytes - 1) / tile_bytes);
  Unit *o = out + (uint64_t)grp * units_per_group + seg_pre[k];
  if (group > 1) {  // runs shorter than a unit: `group` consecutive runs are one unit
    const uint32_t run0 = grp * group, n = n_runs - run0 < group ? n_runs - run0 : group;
    *o = Unit{seg, run0 * tpr, n * tpr, 0};
    return;
  }
  for (uint32_t t = 0; t < tpr; t += unit_tiles, ++o)
    *o = Unit{seg, grp * tpr + t, tpr - t < unit_tiles ? tpr - t : unit_tiles, 0};
}
}  // namespace

cudaError_t launch_gen_units(const DevSeg *segs, const uint32_t *seg_idx, const uint32_t *seg_pre,
                             uint32_t n_segs, uint32_t n_runs, uint32_t group, uint32_t units_per_group,
                             uint32_t tile_bytes, uint32_t unit_tiles, uint32_t seg_offset, Unit *out,
                             cudaStream_t stream) {
  if (group == 0) return cudaErrorInvalidValue;
  const uint64_t n = (uint64_t)n_segs * ((n_runs + group - 1) / group);
  if (n == 0) return cudaSuccess;
  gen_units_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(
      segs, seg_idx, seg_pre, n_segs, n_runs, group, units_per_group, tile_bytes, unit_tiles, seg_offset, out);
  return cudaGetLastError();
}

// ---- KV re-split without any allocation ---------------------------------------------------
//
// For callers that cannot call cudaMalloc (all of HBM already owned by a memory daemon,
// or no tolerance for the implicit synchronisation of an allocation): the block-pair
// list lives in this fixed array of the library image, old ids in the first half, new
// ids in the second.  Every GPU that loads the library holds these 512 KiB until exit.
// In host code the symbol below is only a handle; its device address is looked up once
// per device with cudaGetSymbolAddress and handed to the kernel as an ordinary pointer.
static __device__ __align__(256) uint32_t g_kv_static_pairs[2 * EMOE_STATIC_KV_MAX_PAIRS];

namespace {
std::mutex g_static_mu;
uint32_t *g_static_ptr[kMaxDevices] = {};
int g_static_sms[kMaxDevices] = {};
}  // namespace

emoe_status_t launch_kv_copy_static(const KvTables &shape_only, const uint32_t *pair_old,
                                    const uint32_t *pair_new, const RankPtrs &ptrs,
                                    cudaStream_t stream) {
  const uint32_t n = shape_only.n_pairs;
  if (n > EMOE_STATIC_KV_MAX_PAIRS) return EMOE_ERR_TOO_LARGE;
  if (n == 0 || shape_only.n_lk == 0) return EMOE_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  uint32_t *scratch = nullptr;
  int sms = 0;
  {
    // one-time set-up per device, with that device current
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
      void *p = nullptr;
      if (cudaGetSymbolAddress(&p, g_kv_static_pairs) != cudaSuccess || !p ||
          cudaDeviceGetAttribute(&g_static_sms[dev], cudaDevAttrMultiProcessorCount, dev) !=
              cudaSuccess) {
        (void)cudaGetLastError();
        return EMOE_ERR_CUDA;
      }
      g_static_ptr[dev] = static_cast<uint32_t *>(p);
    }
    scratch = g_static_ptr[dev];
    sms = g_static_sms[dev];
  }
  uint32_t *d_old = scratch, *d_new = scratch + EMOE_STATIC_KV_MAX_PAIRS;
  if (cudaMemcpyAsync(d_old, pair_old, n * sizeof(uint32_t), cudaMemcpyHostToDevice, stream) !=
          cudaSuccess ||
      cudaMemcpyAsync(d_new, pair_new, n * sizeof(uint32_t), cudaMemcpyHostToDevice, stream) !=
          cudaSuccess) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  KvTables t = shape_only;
  t.pair_old = d_old;
  t.pair_new = d_new;
  const cudaError_t e = launch_kv_copy(t, ptrs, 1, (uint32_t)sms, false, nullptr, 0, stream);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return EMOE_ERR_CUDA;
  }
  return EMOE_OK;
}

}  // namespace emoe
