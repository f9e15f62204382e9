// vmm.cpp - paged expert store: expert re-layout by re-mapping pages, copies for arrivals only.
//
// The paper stores every expert in physical pages of its own and maps them into one
// contiguous virtual range per device, so that a change of the expert-parallel degree
// re-maps pages instead of copying tensors (Sec. 4.1 "Virtual Expert Management",
// App. D.5).  This file is that mechanism on the CUDA virtual memory API: one physical
// allocation per expert matrix ("slab": the matrix rounded up to the allocation
// granularity), one reserved virtual range per rank laid out [L][3][n_r][slab].  A scale
// step maps the slabs a rank keeps into its new range (no copy), gives arriving experts
// fresh slabs filled by the bulk copy kernel from their source rank, and releases what no
// range references any more.  On one GPU every rank is a range of that GPU.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cstring>
#include <map>
#include <new>
#include <vector>

#include "internal.h"

using namespace emoe;

namespace {

struct DriverApi {
  CUresult (*MemGetAllocationGranularity)(size_t *, const CUmemAllocationProp *,
                                          CUmemAllocationGranularity_flags) = nullptr;
  CUresult (*MemCreate)(CUmemGenericAllocationHandle *, size_t, const CUmemAllocationProp *,
                        unsigned long long) = nullptr;
  CUresult (*MemRelease)(CUmemGenericAllocationHandle) = nullptr;
  CUresult (*MemAddressReserve)(CUdeviceptr *, size_t, size_t, CUdeviceptr, unsigned long long) = nullptr;
  CUresult (*MemAddressFree)(CUdeviceptr, size_t) = nullptr;
  CUresult (*MemMap)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long) = nullptr;
  CUresult (*MemUnmap)(CUdeviceptr, size_t) = nullptr;
  CUresult (*MemSetAccess)(CUdeviceptr, size_t, const CUmemAccessDesc *, size_t) = nullptr;
  bool ok = false;
};

template <typename F>
bool load_entry(const char *name, F *out) {
  void *p = nullptr;
  cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !p) {
    (void)cudaGetLastError();
    return false;
  }
  *out = reinterpret_cast<F>(p);
  return true;
}

// The driver's virtual memory entry points, looked up through the runtime.
const DriverApi &driver() {
  static DriverApi api = [] {
    DriverApi a;
    a.ok = load_entry("cuMemGetAllocationGranularity", &a.MemGetAllocationGranularity) &&
           load_entry("cuMemCreate", &a.MemCreate) && load_entry("cuMemRelease", &a.MemRelease) &&
           load_entry("cuMemAddressReserve", &a.MemAddressReserve) &&
           load_entry("cuMemAddressFree", &a.MemAddressFree) && load_entry("cuMemMap", &a.MemMap) &&
           load_entry("cuMemUnmap", &a.MemUnmap) && load_entry("cuMemSetAccess", &a.MemSetAccess);
    return a;
  }();
  return api;
}

// One rank's virtual range and the physical slab behind every (layer, projection, slot).
struct Range {
  CUdeviceptr base = 0;
  uint64_t bytes = 0;
  std::vector<CUmemGenericAllocationHandle> slabs;  // index (l*3 + p) * n_slots + slot
  uint32_t n_slots = 0;
  uint64_t mapped = 0;  // slabs mapped so far (for unwinding a failed build)
};

double now_ms() {
  return std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now().time_since_epoch())
      .count();
}

}  // namespace

struct emoe_vmm_pool {
  emoe_shape_t shape{};
  int device = 0;
  uint64_t m = 0, slab = 0;
  uint32_t runs = 0;  // 3 * n_layers
  std::vector<std::vector<int32_t>> placement;
  std::vector<Range> ranges;
  std::map<CUmemGenericAllocationHandle, uint32_t> refs;  // ranges that map the slab
  CUmemAllocationProp prop{};
};

namespace {

void drop_ref(emoe_vmm_pool *pool, CUmemGenericAllocationHandle h) {
  auto it = pool->refs.find(h);
  if (it == pool->refs.end()) return;
  if (--it->second == 0) {
    driver().MemRelease(h);
    pool->refs.erase(it);
  }
}

// Unmaps what a range maps, drops its slab references and frees its address range.
void destroy_range(emoe_vmm_pool *pool, Range *rg) {
  if (!rg->base) return;
  const uint64_t per = pool->slab;
  for (uint64_t i = 0; i < rg->mapped; ++i) {
    driver().MemUnmap(rg->base + i * per, per);
    drop_ref(pool, rg->slabs[i]);
  }
  driver().MemAddressFree(rg->base, rg->bytes);
  rg->base = 0;
  rg->mapped = 0;
}

emoe_status_t reserve_range(const emoe_vmm_pool *pool, uint32_t n_slots, Range *rg) {
  rg->n_slots = n_slots;
  rg->bytes = (uint64_t)pool->runs * n_slots * pool->slab;
  rg->slabs.assign((size_t)pool->runs * n_slots, 0);
  rg->mapped = 0;
  rg->base = 0;
  if (!rg->bytes) return EMOE_OK;
  // default alignment (the allocation granularity): a slab size need not be a power of two
  const CUresult r = driver().MemAddressReserve(&rg->base, rg->bytes, 0, 0, 0);
  if (r != CUDA_SUCCESS) {
    rg->base = 0;
    return r == CUDA_ERROR_OUT_OF_MEMORY ? EMOE_ERR_OOM : EMOE_ERR_CUDA;
  }
  return EMOE_OK;
}

// Maps `h` as the next slab of the range (slabs are mapped in index order).
emoe_status_t map_next(emoe_vmm_pool *pool, Range *rg, CUmemGenericAllocationHandle h) {
  const uint64_t i = rg->mapped;
  if (driver().MemMap(rg->base + i * pool->slab, pool->slab, 0, h, 0) != CUDA_SUCCESS) return EMOE_ERR_CUDA;
  rg->slabs[i] = h;
  rg->mapped = i + 1;
  pool->refs[h]++;
  return EMOE_OK;
}

emoe_status_t new_slab(emoe_vmm_pool *pool, CUmemGenericAllocationHandle *h) {
  const CUresult r = driver().MemCreate(h, pool->slab, &pool->prop, 0);
  if (r == CUDA_ERROR_OUT_OF_MEMORY) return EMOE_ERR_OOM;
  return r == CUDA_SUCCESS ? EMOE_OK : EMOE_ERR_CUDA;
}

emoe_status_t enable_access(const emoe_vmm_pool *pool, const Range &rg) {
  if (!rg.bytes) return EMOE_OK;
  CUmemAccessDesc d{};
  d.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
  d.location.id = pool->device;
  d.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
  return driver().MemSetAccess(rg.base, rg.bytes, &d, 1) == CUDA_SUCCESS ? EMOE_OK : EMOE_ERR_CUDA;
}

emoe_status_t read_ids(const emoe_shape_t &sh, const emoe_config_t &cfg,
                       std::vector<std::vector<int32_t>> *out) {
  // validated by the planner before this is called
  (void)sh;
  out->assign(cfg.ep, {});
  for (int r = 0; r < cfg.ep; ++r)
    for (int i = cfg.place_off[r]; i < cfg.place_off[r + 1]; ++i) (*out)[r].push_back(cfg.place_ids[i]);
  return EMOE_OK;
}

}  // namespace

extern "C" {

emoe_status_t emoe_vmm_create(const emoe_shape_t *shape, const emoe_config_t *cfg,
                              emoe_vmm_pool_t **out) {
  if (!shape || !cfg || !out) return EMOE_ERR_INVALID_ARG;
  // validation of shape and placement: plan the identity step
  try {
    PhasePlan pp;
    const uint64_t m = (uint64_t)shape->d_model * shape->d_ff * shape->elem_bytes;
    emoe_status_t st = build_paged_expert_plan(*shape, *cfg, *cfg, m > 0 ? m : 1, &pp, nullptr);
    if (st != EMOE_OK) return st;
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  if (cudaFree(nullptr) != cudaSuccess) { (void)cudaGetLastError(); return EMOE_ERR_CUDA; }
  if (!driver().ok) return EMOE_ERR_UNSUPPORTED;
  emoe_vmm_pool *pool = new (std::nothrow) emoe_vmm_pool();
  if (!pool) return EMOE_ERR_OOM;
  emoe_status_t st = EMOE_OK;
  try {
    pool->shape = *shape;
    if (cudaGetDevice(&pool->device) != cudaSuccess) { delete pool; return EMOE_ERR_CUDA; }
    pool->prop.type = CU_MEM_ALLOCATION_TYPE_PINNED;
    pool->prop.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    pool->prop.location.id = pool->device;
    size_t gran = 0;
    if (driver().MemGetAllocationGranularity(&gran, &pool->prop, CU_MEM_ALLOC_GRANULARITY_MINIMUM) !=
            CUDA_SUCCESS || gran == 0) {
      delete pool;
      return EMOE_ERR_UNSUPPORTED;
    }
    pool->m = (uint64_t)shape->d_model * shape->d_ff * shape->elem_bytes;
    pool->slab = (pool->m + gran - 1) / gran * gran;
    pool->runs = 3u * (uint32_t)shape->n_layers;
    read_ids(*shape, *cfg, &pool->placement);
    pool->ranges.resize(cfg->ep);
    for (int r = 0; st == EMOE_OK && r < cfg->ep; ++r) {
      Range &rg = pool->ranges[r];
      st = reserve_range(pool, (uint32_t)pool->placement[r].size(), &rg);
      for (size_t i = 0; st == EMOE_OK && i < rg.slabs.size(); ++i) {
        CUmemGenericAllocationHandle h = 0;
        st = new_slab(pool, &h);
        if (st != EMOE_OK) break;
        st = map_next(pool, &rg, h);
        if (st != EMOE_OK) driver().MemRelease(h);
      }
      if (st == EMOE_OK) st = enable_access(pool, rg);
    }
  } catch (const std::bad_alloc &) {
    st = EMOE_ERR_OOM;
  }
  if (st != EMOE_OK) {
    emoe_vmm_destroy(pool);
    return st;
  }
  *out = pool;
  return EMOE_OK;
}

void emoe_vmm_destroy(emoe_vmm_pool_t *pool) {
  if (!pool) return;
  (void)cudaDeviceSynchronize();
  for (Range &rg : pool->ranges) destroy_range(pool, &rg);
  delete pool;
}

emoe_status_t emoe_vmm_num_ranks(const emoe_vmm_pool_t *pool, int32_t *n) {
  if (!pool || !n) return EMOE_ERR_INVALID_ARG;
  *n = (int32_t)pool->ranges.size();
  return EMOE_OK;
}

emoe_status_t emoe_vmm_arena(const emoe_vmm_pool_t *pool, int rank, void **base, uint64_t *bytes,
                             uint64_t *slab_bytes, uint64_t *matrix_bytes, int32_t *n_slots) {
  if (!pool || rank < 0 || rank >= (int)pool->ranges.size()) return EMOE_ERR_INVALID_ARG;
  const Range &rg = pool->ranges[rank];
  if (base) *base = reinterpret_cast<void *>(rg.base);
  if (bytes) *bytes = rg.bytes;
  if (slab_bytes) *slab_bytes = pool->slab;
  if (matrix_bytes) *matrix_bytes = pool->m;
  if (n_slots) *n_slots = (int32_t)rg.n_slots;
  return EMOE_OK;
}

// Dense host image [L][3][n_r][m] <-> the rank's paged range (rows of m bytes, slab apart).
emoe_status_t emoe_vmm_write(emoe_vmm_pool_t *pool, int rank, const void *host_dense, void *stream) {
  if (!pool || rank < 0 || rank >= (int)pool->ranges.size() || !host_dense) return EMOE_ERR_INVALID_ARG;
  const Range &rg = pool->ranges[rank];
  if (!rg.bytes) return EMOE_OK;
  const cudaError_t e = cudaMemcpy2DAsync(reinterpret_cast<void *>(rg.base), pool->slab, host_dense, pool->m,
                                          pool->m, rg.slabs.size(), cudaMemcpyHostToDevice,
                                          (cudaStream_t)stream);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return EMOE_ERR_CUDA; }
  return EMOE_OK;
}

emoe_status_t emoe_vmm_read(const emoe_vmm_pool_t *pool, int rank, void *host_dense, void *stream) {
  if (!pool || rank < 0 || rank >= (int)pool->ranges.size() || !host_dense) return EMOE_ERR_INVALID_ARG;
  const Range &rg = pool->ranges[rank];
  if (!rg.bytes) return EMOE_OK;
  const cudaError_t e = cudaMemcpy2DAsync(host_dense, pool->m, reinterpret_cast<const void *>(rg.base),
                                          pool->slab, pool->m, rg.slabs.size(), cudaMemcpyDeviceToHost,
                                          (cudaStream_t)stream);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return EMOE_ERR_CUDA; }
  return EMOE_OK;
}

emoe_status_t emoe_vmm_dry_run(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                               const emoe_config_t *new_cfg, uint64_t slab_bytes,
                               emoe_vmm_stats_t *stats) {
  if (!shape || !old_cfg || !new_cfg || !stats) return EMOE_ERR_INVALID_ARG;
  try {
    PhasePlan pp;
    std::vector<Remap> remaps;
    emoe_config_t o = *old_cfg, n = *new_cfg;
    if (o.tp < 1) o.tp = 1;
    if (n.tp < 1) n.tp = 1;
    const emoe_status_t st = build_paged_expert_plan(*shape, o, n, slab_bytes, &pp, &remaps);
    if (st != EMOE_OK) return st;
    emoe_vmm_stats_t s{};
    const uint64_t runs = 3ull * (uint64_t)shape->n_layers;
    const uint64_t slots = (uint64_t)n.place_off[n.ep];
    s.slabs_remapped = remaps.size() * runs;
    s.slabs_copied = (slots - remaps.size()) * runs;
    s.bytes_copied = pp.bytes_moved;
    s.bytes_read = pp.bytes_read;
    s.slab_bytes = slab_bytes;
    s.matrix_bytes = (uint64_t)shape->d_model * shape->d_ff * shape->elem_bytes;
    s.physical_bytes = slots * runs * slab_bytes;
    *stats = s;
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}

emoe_status_t emoe_vmm_reshard(emoe_vmm_pool_t *pool, const emoe_config_t *new_cfg, void *stream,
                               emoe_vmm_stats_t *stats) {
  if (!pool || !new_cfg) return EMOE_ERR_INVALID_ARG;
  if (new_cfg->ep < 1 || new_cfg->ep > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  emoe_vmm_stats_t s{};
  const double t0 = now_ms();
  emoe_status_t rc = EMOE_OK;
  std::vector<Range> fresh;
  try {
    // the pool's current placement as a configuration
    std::vector<int32_t> off(pool->placement.size() + 1, 0), ids;
    for (size_t r = 0; r < pool->placement.size(); ++r) {
      off[r + 1] = off[r] + (int32_t)pool->placement[r].size();
      ids.insert(ids.end(), pool->placement[r].begin(), pool->placement[r].end());
    }
    if (ids.empty()) ids.push_back(0);
    emoe_config_t old_cfg{};
    old_cfg.ep = (int32_t)pool->placement.size();
    old_cfg.tp = 1;
    old_cfg.place_off = off.data();
    old_cfg.place_ids = ids.data();
    emoe_config_t ncfg = *new_cfg;
    if (ncfg.tp < 1) ncfg.tp = 1;

    PhasePlan pp;
    std::vector<Remap> remaps;
    rc = build_paged_expert_plan(pool->shape, old_cfg, ncfg, pool->slab, &pp, &remaps);
    if (rc != EMOE_OK) return rc;
    std::vector<std::vector<int32_t>> new_ids;
    read_ids(pool->shape, ncfg, &new_ids);

    // which old slot every kept destination slot re-uses (rank index is the same)
    std::vector<std::vector<int32_t>> keep(new_ids.size());
    for (size_t r = 0; r < new_ids.size(); ++r) keep[r].assign(new_ids[r].size(), -1);
    for (const Remap &mp : remaps) keep[mp.dst_rank][mp.dst_slot] = (int32_t)mp.src_slot;

    // new ranges: kept slabs are mapped a second time, arrivals get fresh slabs
    fresh.resize(new_ids.size());
    for (size_t r = 0; rc == EMOE_OK && r < new_ids.size(); ++r) {
      Range &rg = fresh[r];
      rc = reserve_range(pool, (uint32_t)new_ids[r].size(), &rg);
      const uint32_t n_new = rg.n_slots;
      for (uint32_t run = 0; rc == EMOE_OK && run < pool->runs; ++run)
        for (uint32_t sd = 0; rc == EMOE_OK && sd < n_new; ++sd) {
          const int32_t ss = keep[r][sd];
          if (ss >= 0) {
            const Range &old = pool->ranges[r];
            rc = map_next(pool, &rg, old.slabs[(size_t)run * old.n_slots + ss]);
            s.slabs_remapped++;
          } else {
            CUmemGenericAllocationHandle h = 0;
            const double ta = now_ms();
            rc = new_slab(pool, &h);
            s.alloc_ms += now_ms() - ta;
            if (rc != EMOE_OK) break;
            rc = map_next(pool, &rg, h);
            if (rc != EMOE_OK) driver().MemRelease(h);
            s.slabs_copied++;
          }
        }
      const double ta = now_ms();
      if (rc == EMOE_OK) rc = enable_access(pool, rg);
      s.access_ms += now_ms() - ta;
    }
    const double t1 = now_ms();
    s.map_ms = t1 - t0;

    // arrivals: the copy kernels read the old ranges and write the new ones
    if (rc == EMOE_OK && !pp.segs.empty()) {
      RankPtrs ptrs;
      std::memset(&ptrs, 0, sizeof(ptrs));
      for (size_t r = 0; r < pool->ranges.size(); ++r)
        ptrs.src[r] = reinterpret_cast<const uint8_t *>(pool->ranges[r].base);
      for (size_t r = 0; r < fresh.size(); ++r) ptrs.dst[r] = reinterpret_cast<uint8_t *>(fresh[r].base);
      rc = run_phase_once(pp, ptrs, st);
      s.bytes_copied = pp.bytes_moved;
      s.bytes_read = pp.bytes_read;
    } else if (rc == EMOE_OK) {
      if (cudaStreamSynchronize(st) != cudaSuccess) { (void)cudaGetLastError(); rc = EMOE_ERR_CUDA; }
    }
    const double t2 = now_ms();
    s.copy_ms = t2 - t1;
    if (rc != EMOE_OK) {
      for (Range &rg : fresh) destroy_range(pool, &rg);
      return rc;
    }
    // retire the old ranges; slabs no range maps any more are released
    for (Range &rg : pool->ranges) destroy_range(pool, &rg);
    pool->ranges = std::move(fresh);
    pool->placement = std::move(new_ids);
    s.unmap_ms = now_ms() - t2;
  } catch (const std::bad_alloc &) {
    for (Range &rg : fresh) destroy_range(pool, &rg);
    return EMOE_ERR_OOM;
  }
  s.total_ms = now_ms() - t0;
  s.slab_bytes = pool->slab;
  s.matrix_bytes = pool->m;
  s.physical_bytes = (uint64_t)pool->refs.size() * pool->slab;
  if (stats) *stats = s;
  return EMOE_OK;
}

}  // extern "C"

// ---- paged store with slot tables: a step touches only the slots that change ------------
//
// The store above rebuilds every range at every step.  This one keeps a device's range for
// as long as the device exists: the range is RESERVED for `cap` slots per (layer,
// projection), [L][3][cap][slab], and only occupied slots have pages behind them.  A step
// follows the in-place expert step (emoe_plan_create_inplace): kept experts are not
// touched at all, an arrival gets pages mapped into a slot that was free before the step
// and is filled by the copy kernels, a leaving expert's pages are unmapped AFTER the copies
// and go back to a list of spare pages, from which later arrivals are served - so that, in
// the steady state, a step neither creates nor releases physical memory and its driver work
// is proportional to the slots that change.

namespace {

struct SlotRange {
  CUdeviceptr base = 0;
  uint64_t bytes = 0;
  uint32_t cap = 0;
  std::vector<int32_t> ids;                          // expert per slot, -1 free
  std::vector<CUmemGenericAllocationHandle> slabs;   // index run * cap + slot; 0 = nothing mapped
};

}  // namespace

struct emoe_vmm_slots {
  emoe_shape_t shape{};
  int device = 0;
  uint64_t m = 0, slab = 0;
  uint32_t runs = 0;
  std::vector<SlotRange> ranges;
  std::vector<CUmemGenericAllocationHandle> spare;   // physical slabs that no slot maps
  CUmemAllocationProp prop{};
  CUmemAccessDesc access{};
};

namespace {

CUdeviceptr slot_addr(const emoe_vmm_slots *pool, const SlotRange &rg, uint32_t run, uint32_t slot) {
  return rg.base + ((uint64_t)run * rg.cap + slot) * pool->slab;
}

emoe_status_t take_slab(emoe_vmm_slots *pool, CUmemGenericAllocationHandle *h, double *alloc_ms) {
  if (!pool->spare.empty()) {
    *h = pool->spare.back();
    pool->spare.pop_back();
    return EMOE_OK;
  }
  const double t = now_ms();
  const CUresult r = driver().MemCreate(h, pool->slab, &pool->prop, 0);
  if (alloc_ms) *alloc_ms += now_ms() - t;
  if (r == CUDA_ERROR_OUT_OF_MEMORY) return EMOE_ERR_OOM;
  return r == CUDA_SUCCESS ? EMOE_OK : EMOE_ERR_CUDA;
}

// Pages behind every (layer, projection) of one slot.  On failure what was mapped stays
// recorded in rg.slabs, so that unmap_slot / the destructor undo it.
emoe_status_t map_slot(emoe_vmm_slots *pool, SlotRange *rg, uint32_t slot, double *alloc_ms, double *access_ms) {
  for (uint32_t run = 0; run < pool->runs; ++run) {
    CUmemGenericAllocationHandle h = 0;
    emoe_status_t st = take_slab(pool, &h, alloc_ms);
    if (st != EMOE_OK) return st;
    const CUdeviceptr at = slot_addr(pool, *rg, run, slot);
    if (driver().MemMap(at, pool->slab, 0, h, 0) != CUDA_SUCCESS) {
      pool->spare.push_back(h);
      return EMOE_ERR_CUDA;
    }
    rg->slabs[(size_t)run * rg->cap + slot] = h;
  }
  (void)access_ms;
  return EMOE_OK;
}

// Enables access to freshly mapped slots: one driver call per (layer, projection) and per run
// of neighbouring slots, since neighbouring slots are neighbours in the address range.
emoe_status_t enable_slots(emoe_vmm_slots *pool, const SlotRange &rg, const std::vector<uint32_t> &slots,
                           double *access_ms) {
  const double t = now_ms();
  emoe_status_t st = EMOE_OK;
  for (uint32_t run = 0; st == EMOE_OK && run < pool->runs; ++run) {
    size_t i = 0;
    while (st == EMOE_OK && i < slots.size()) {
      size_t j = i + 1;
      while (j < slots.size() && slots[j] == slots[j - 1] + 1) ++j;
      if (driver().MemSetAccess(slot_addr(pool, rg, run, slots[i]), (j - i) * pool->slab, &pool->access, 1) !=
          CUDA_SUCCESS)
        st = EMOE_ERR_CUDA;
      i = j;
    }
  }
  if (access_ms) *access_ms += now_ms() - t;
  return st;
}

void unmap_slot(emoe_vmm_slots *pool, SlotRange *rg, uint32_t slot) {
  for (uint32_t run = 0; run < pool->runs; ++run) {
    CUmemGenericAllocationHandle &h = rg->slabs[(size_t)run * rg->cap + slot];
    if (!h) continue;
    driver().MemUnmap(slot_addr(pool, *rg, run, slot), pool->slab);
    pool->spare.push_back(h);
    h = 0;
  }
}

emoe_status_t reserve_slots(emoe_vmm_slots *pool, uint32_t cap, SlotRange *rg) {
  rg->cap = cap;
  rg->bytes = (uint64_t)pool->runs * cap * pool->slab;
  rg->ids.assign(cap, -1);
  rg->slabs.assign((size_t)pool->runs * cap, 0);
  rg->base = 0;
  if (!rg->bytes) return EMOE_OK;
  const CUresult r = driver().MemAddressReserve(&rg->base, rg->bytes, 0, 0, 0);
  if (r != CUDA_SUCCESS) {
    rg->base = 0;
    return r == CUDA_ERROR_OUT_OF_MEMORY ? EMOE_ERR_OOM : EMOE_ERR_CUDA;
  }
  return EMOE_OK;
}

void drop_range(emoe_vmm_slots *pool, SlotRange *rg) {
  if (!rg->base) return;
  for (uint32_t s = 0; s < rg->cap; ++s) unmap_slot(pool, rg, s);
  driver().MemAddressFree(rg->base, rg->bytes);
  rg->base = 0;
}

}  // namespace

extern "C" {

emoe_status_t emoe_vmm_slots_create(const emoe_shape_t *shape, int32_t ep, const int32_t *slot_off,
                                    const int32_t *slot_ids, int32_t spare_slots,
                                    emoe_vmm_slots_t **out) {
  if (!shape || !slot_off || !slot_ids || !out || ep < 1 || spare_slots < 0) return EMOE_ERR_INVALID_ARG;
  if (ep > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  try {  // validation of shape and tables: plan the step that changes nothing
    PhasePlan pp;
    std::vector<std::vector<int32_t>> tables;
    std::vector<int32_t> cap(ep), want_off(ep + 1, 0), want;
    for (int r = 0; r < ep; ++r) {
      if (slot_off[r + 1] < slot_off[r]) return EMOE_ERR_PLACEMENT;
      cap[r] = slot_off[r + 1] - slot_off[r];
      for (int i = slot_off[r]; i < slot_off[r + 1]; ++i)
        if (slot_ids[i] >= 0) want.push_back(slot_ids[i]);
      want_off[r + 1] = (int32_t)want.size();
    }
    if (want.empty()) want.push_back(0);
    const emoe_status_t st = build_inplace_expert_plan(*shape, ep, slot_off, slot_ids, ep, cap.data(),
                                                       want_off.data(), want.data(), 0, &pp, &tables);
    if (st != EMOE_OK) return st;
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  if (cudaFree(nullptr) != cudaSuccess) { (void)cudaGetLastError(); return EMOE_ERR_CUDA; }
  if (!driver().ok) return EMOE_ERR_UNSUPPORTED;
  emoe_vmm_slots *pool = new (std::nothrow) emoe_vmm_slots();
  if (!pool) return EMOE_ERR_OOM;
  emoe_status_t st = EMOE_OK;
  try {
    pool->shape = *shape;
    if (cudaGetDevice(&pool->device) != cudaSuccess) { delete pool; return EMOE_ERR_CUDA; }
    pool->prop.type = CU_MEM_ALLOCATION_TYPE_PINNED;
    pool->prop.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    pool->prop.location.id = pool->device;
    pool->access.location = pool->prop.location;
    pool->access.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
    size_t gran = 0;
    if (driver().MemGetAllocationGranularity(&gran, &pool->prop, CU_MEM_ALLOC_GRANULARITY_MINIMUM) !=
            CUDA_SUCCESS || gran == 0) {
      delete pool;
      return EMOE_ERR_UNSUPPORTED;
    }
    pool->m = (uint64_t)shape->d_model * shape->d_ff * shape->elem_bytes;
    pool->slab = (pool->m + gran - 1) / gran * gran;
    pool->runs = 3u * (uint32_t)shape->n_layers;
    pool->ranges.resize(ep);
    for (int r = 0; st == EMOE_OK && r < ep; ++r) {
      SlotRange &rg = pool->ranges[r];
      st = reserve_slots(pool, (uint32_t)(slot_off[r + 1] - slot_off[r]), &rg);
      std::vector<uint32_t> mapped;
      for (uint32_t s = 0; st == EMOE_OK && s < rg.cap; ++s) {
        rg.ids[s] = slot_ids[slot_off[r] + s];
        if (rg.ids[s] >= 0) {
          st = map_slot(pool, &rg, s, nullptr, nullptr);
          mapped.push_back(s);
        }
      }
      if (st == EMOE_OK) st = enable_slots(pool, rg, mapped, nullptr);
    }
    // spare pages for the arrivals of later steps: created now, outside any step
    for (int64_t i = 0; st == EMOE_OK && i < (int64_t)spare_slots * pool->runs; ++i) {
      CUmemGenericAllocationHandle h = 0;
      const CUresult r = driver().MemCreate(&h, pool->slab, &pool->prop, 0);
      if (r != CUDA_SUCCESS) { st = r == CUDA_ERROR_OUT_OF_MEMORY ? EMOE_ERR_OOM : EMOE_ERR_CUDA; break; }
      pool->spare.push_back(h);
    }
  } catch (const std::bad_alloc &) {
    st = EMOE_ERR_OOM;
  }
  if (st != EMOE_OK) {
    emoe_vmm_slots_destroy(pool);
    return st;
  }
  *out = pool;
  return EMOE_OK;
}

void emoe_vmm_slots_destroy(emoe_vmm_slots_t *pool) {
  if (!pool) return;
  (void)cudaDeviceSynchronize();
  for (SlotRange &rg : pool->ranges) drop_range(pool, &rg);
  for (CUmemGenericAllocationHandle h : pool->spare) driver().MemRelease(h);
  delete pool;
}

emoe_status_t emoe_vmm_slots_info(const emoe_vmm_slots_t *pool, int32_t rank, void **base,
                                  uint64_t *slab_bytes, int32_t *cap, int32_t *ids_out, int32_t ids_cap,
                                  int32_t *n_ranks, int64_t *spare_slabs) {
  if (!pool) return EMOE_ERR_INVALID_ARG;
  if (n_ranks) *n_ranks = (int32_t)pool->ranges.size();
  if (spare_slabs) *spare_slabs = (int64_t)pool->spare.size();
  if (slab_bytes) *slab_bytes = pool->slab;
  if (rank < 0) return EMOE_OK;                       // pool-wide figures only
  if (rank >= (int)pool->ranges.size() || (ids_cap > 0 && !ids_out)) return EMOE_ERR_INVALID_ARG;
  const SlotRange &rg = pool->ranges[rank];
  if (base) *base = reinterpret_cast<void *>(rg.base);
  if (cap) *cap = (int32_t)rg.cap;
  for (int32_t i = 0; i < ids_cap && i < (int32_t)rg.cap; ++i) ids_out[i] = rg.ids[i];
  return EMOE_OK;
}

// One slot as a dense host image [L][3][m] <-> its pages.  One copy per (layer, projection):
// the rows of a slot are a whole layer slab apart and what lies between them may be unmapped,
// which a strided 2-D copy does not accept.
emoe_status_t emoe_vmm_slots_write(emoe_vmm_slots_t *pool, int32_t rank, int32_t slot, const void *host,
                                   void *stream) {
  if (!pool || rank < 0 || rank >= (int)pool->ranges.size() || !host) return EMOE_ERR_INVALID_ARG;
  const SlotRange &rg = pool->ranges[rank];
  if (slot < 0 || slot >= (int)rg.cap || rg.ids[slot] < 0) return EMOE_ERR_INVALID_ARG;
  for (uint32_t run = 0; run < pool->runs; ++run)
    if (cudaMemcpyAsync(reinterpret_cast<void *>(slot_addr(pool, rg, run, (uint32_t)slot)),
                        static_cast<const uint8_t *>(host) + (uint64_t)run * pool->m, pool->m,
                        cudaMemcpyHostToDevice, (cudaStream_t)stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return EMOE_ERR_CUDA;
    }
  return EMOE_OK;
}

emoe_status_t emoe_vmm_slots_read(const emoe_vmm_slots_t *pool, int32_t rank, int32_t slot, void *host,
                                  void *stream) {
  if (!pool || rank < 0 || rank >= (int)pool->ranges.size() || !host) return EMOE_ERR_INVALID_ARG;
  const SlotRange &rg = pool->ranges[rank];
  if (slot < 0 || slot >= (int)rg.cap || rg.ids[slot] < 0) return EMOE_ERR_INVALID_ARG;
  for (uint32_t run = 0; run < pool->runs; ++run)
    if (cudaMemcpyAsync(static_cast<uint8_t *>(host) + (uint64_t)run * pool->m,
                        reinterpret_cast<const void *>(slot_addr(pool, rg, run, (uint32_t)slot)), pool->m,
                        cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return EMOE_ERR_CUDA;
    }
  return EMOE_OK;
}

emoe_status_t emoe_vmm_slots_reshard(emoe_vmm_slots_t *pool, int32_t ep_new, const int32_t *cap_new,
                                     const int32_t *want_off, const int32_t *want_ids, void *stream,
                                     emoe_vmm_stats_t *stats) {
  if (!pool || !cap_new || !want_off || !want_ids) return EMOE_ERR_INVALID_ARG;
  if (ep_new < 1 || ep_new > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  emoe_vmm_stats_t s{};
  const double t0 = now_ms();
  emoe_status_t rc = EMOE_OK;
  const int ep_old = (int)pool->ranges.size();
  try {
    std::vector<int32_t> off(ep_old + 1, 0), ids;
    for (int r = 0; r < ep_old; ++r) {
      off[r + 1] = off[r] + (int32_t)pool->ranges[r].cap;
      ids.insert(ids.end(), pool->ranges[r].ids.begin(), pool->ranges[r].ids.end());
    }
    if (ids.empty()) ids.push_back(-1);
    PhasePlan pp;
    std::vector<std::vector<int32_t>> slot_new;
    rc = build_inplace_expert_plan(pool->shape, ep_old, off.data(), ids.data(), ep_new, cap_new, want_off,
                                   want_ids, pool->slab, &pp, &slot_new);
    if (rc != EMOE_OK) return rc;            // nothing has been touched yet

    // 1. ranges of added devices, pages behind every arrival's slot
    const size_t n_dev = (size_t)std::max(ep_old, (int)ep_new);
    if (pool->ranges.size() < n_dev) pool->ranges.resize(n_dev);
    std::vector<std::pair<int, uint32_t>> arrived;    // (rank, slot) mapped by this step
    for (int r = 0; rc == EMOE_OK && r < ep_new; ++r) {
      SlotRange &rg = pool->ranges[r];
      if (r >= ep_old) rc = reserve_slots(pool, (uint32_t)cap_new[r], &rg);
      std::vector<uint32_t> mine;
      for (uint32_t sl = 0; rc == EMOE_OK && sl < rg.cap; ++sl) {
        const int32_t e = slot_new[r][sl];
        if (e < 0 || (r < ep_old && rg.ids[sl] == e)) continue;   // free, or kept: not touched
        arrived.push_back({r, sl});
        mine.push_back(sl);
        rc = map_slot(pool, &rg, sl, &s.alloc_ms, &s.access_ms);
        s.slabs_copied += pool->runs;
      }
      if (rc == EMOE_OK) rc = enable_slots(pool, rg, mine, &s.access_ms);
    }
    const double t1 = now_ms();
    s.map_ms = t1 - t0;

    // 2. the copy kernels fill the arrivals from their sources (ranges as they are now)
    if (rc == EMOE_OK && !pp.segs.empty()) {
      RankPtrs ptrs;
      std::memset(&ptrs, 0, sizeof(ptrs));
      for (int r = 0; r < ep_old; ++r) ptrs.src[r] = reinterpret_cast<const uint8_t *>(pool->ranges[r].base);
      for (int r = 0; r < ep_new; ++r) ptrs.dst[r] = reinterpret_cast<uint8_t *>(pool->ranges[r].base);
      rc = run_phase_once(pp, ptrs, st);
      s.bytes_copied = pp.bytes_moved;
      s.bytes_read = pp.bytes_read;
    } else if (rc == EMOE_OK) {
      if (cudaStreamSynchronize(st) != cudaSuccess) { (void)cudaGetLastError(); rc = EMOE_ERR_CUDA; }
    }
    const double t2 = now_ms();
    s.copy_ms = t2 - t1;
    if (rc != EMOE_OK) {   // undo: the pool is as it was before the call
      for (auto &a : arrived) unmap_slot(pool, &pool->ranges[a.first], a.second);
      for (size_t r = ep_old; r < pool->ranges.size(); ++r) drop_range(pool, &pool->ranges[r]);
      pool->ranges.resize(ep_old);
      return rc;
    }

    // 3. experts that left: their pages go back to the spare list; removed devices go whole
    for (int r = 0; r < ep_old; ++r) {
      SlotRange &rg = pool->ranges[r];
      if (r >= ep_new) { drop_range(pool, &rg); continue; }
      for (uint32_t sl = 0; sl < rg.cap; ++sl)
        if (rg.ids[sl] >= 0 && slot_new[r][sl] != rg.ids[sl]) unmap_slot(pool, &rg, sl);
    }
    pool->ranges.resize(ep_new);
    uint64_t kept = 0;
    for (int r = 0; r < ep_new; ++r) {
      for (uint32_t sl = 0; sl < pool->ranges[r].cap; ++sl)
        if (slot_new[r][sl] >= 0 && r < ep_old && pool->ranges[r].ids[sl] == slot_new[r][sl]) ++kept;
      pool->ranges[r].ids = slot_new[r];
    }
    s.slabs_remapped = kept * pool->runs;      // kept in place: no driver call at all
    s.unmap_ms = now_ms() - t2;
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  s.total_ms = now_ms() - t0;
  s.slab_bytes = pool->slab;
  s.matrix_bytes = pool->m;
  uint64_t mapped = 0;
  for (const SlotRange &rg : pool->ranges)
    for (CUmemGenericAllocationHandle h : rg.slabs) mapped += h != 0;
  s.physical_bytes = (mapped + pool->spare.size()) * pool->slab;
  if (stats) *stats = s;
  return EMOE_OK;
}

}  // extern "C"

