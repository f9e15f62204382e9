// cache.cpp - plan cache for scaling sequences, and the compacting KV block table.
//
// A serving system that scales up and down keeps meeting the same (old, new) pairs of
// configurations (the paper's step patterns add or remove two devices at a time, Sec. 7.4,
// and scale-down mirrors scale-up, App. E).  A plan is a pure function of the model shape,
// the two configurations and the flags, so it can be kept and reused; only plans whose
// inputs are byte-for-byte the same are shared.
#include <cuda_runtime_api.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <list>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/emoe.h"

namespace {

void put(std::string *k, const void *p, size_t n) { k->append(static_cast<const char *>(p), n); }
void put_i32(std::string *k, int32_t v) { put(k, &v, sizeof(v)); }

// Everything emoe_plan_create reads from a configuration, serialised.  Returns false if a
// pointer it would have to follow is null or a count is negative (the planner then reports
// the proper error; such inputs are never cached).
bool config_key(const emoe_shape_t &sh, const emoe_config_t &c, std::string *k) {
  put_i32(k, c.ep); put_i32(k, c.tp); put_i32(k, c.kv_num_blocks); put_i32(k, c.n_seqs);
  if (c.ep < 1 || c.ep > EMOE_MAX_RANKS || !c.place_off || !c.place_ids || c.n_seqs < 0) return false;
  if (c.place_off[0] != 0) return false;
  for (int r = 0; r < c.ep; ++r)
    if (c.place_off[r + 1] < c.place_off[r]) return false;
  put(k, c.place_off, sizeof(int32_t) * (c.ep + 1));
  put(k, c.place_ids, sizeof(int32_t) * c.place_off[c.ep]);
  if (c.n_seqs == 0) return true;
  if (!c.seq_lens || !c.block_table || c.max_blocks < 0 || sh.kv_block_tokens <= 0) return false;
  put(k, c.seq_lens, sizeof(int32_t) * c.n_seqs);
  for (int s = 0; s < c.n_seqs; ++s) {   // only the entries a plan reads: padding may differ
    if (c.seq_lens[s] < 0) return false;
    const int64_t n = ((int64_t)c.seq_lens[s] + sh.kv_block_tokens - 1) / sh.kv_block_tokens;
    if (n > c.max_blocks) return false;
    put(k, c.block_table + (int64_t)s * c.max_blocks, sizeof(int32_t) * n);
    put_i32(k, -1);
  }
  return true;
}

struct Entry {
  std::string key;
  emoe_plan_t *plan;
};

}  // namespace

struct emoe_plan_cache {
  std::mutex mu;
  std::list<Entry> lru;  // most recently used first
  size_t capacity = 0;
  uint64_t hits = 0, misses = 0, evictions = 0;
};

extern "C" {

emoe_status_t emoe_plan_cache_create(int32_t capacity, emoe_plan_cache_t **out) {
  if (!out || capacity < 1) return EMOE_ERR_INVALID_ARG;
  emoe_plan_cache *c = new (std::nothrow) emoe_plan_cache();
  if (!c) return EMOE_ERR_OOM;
  c->capacity = (size_t)capacity;
  *out = c;
  return EMOE_OK;
}

emoe_status_t emoe_plan_cache_get(emoe_plan_cache_t *c, const emoe_shape_t *shape,
                                  const emoe_config_t *old_cfg, const emoe_config_t *new_cfg,
                                  uint32_t flags, const emoe_plan_options_t *options,
                                  emoe_plan_t **plan, int32_t *hit) {
  if (!c || !shape || !old_cfg || !new_cfg || !plan) return EMOE_ERR_INVALID_ARG;
  std::string key;
  bool cacheable = true;
  try {
    put(&key, shape, sizeof(*shape));
    put(&key, &flags, sizeof(flags));
    const int64_t scale = options ? options->expert_scale_bytes : 0;
    const int64_t replicas = options ? options->attn_new_replicas : 0;
    put(&key, &scale, sizeof(scale));
    put(&key, &replicas, sizeof(replicas));
    // a plan's tables live on the device that was current when it was made
    int device = -1;
    if (!(flags & EMOE_PLAN_HOST_ONLY) && cudaGetDevice(&device) != cudaSuccess) device = -1;
    put_i32(&key, device);
    cacheable = config_key(*shape, *old_cfg, &key) && config_key(*shape, *new_cfg, &key);
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  std::lock_guard<std::mutex> lock(c->mu);
  if (cacheable)
    for (auto it = c->lru.begin(); it != c->lru.end(); ++it)
      if (!it->key.empty() && it->key == key) {
        c->lru.splice(c->lru.begin(), c->lru, it);
        ++c->hits;
        *plan = c->lru.front().plan;
        if (hit) *hit = 1;
        return EMOE_OK;
      }
  emoe_plan_t *p = nullptr;
  const emoe_status_t st = emoe_plan_create_ex(shape, old_cfg, new_cfg, flags, options, &p);
  if (st != EMOE_OK) return st;   // invalid inputs are reported, never stored
  ++c->misses;
  // An input the planner accepts although its key could not be formed completely is owned
  // and evicted like any other plan but never found again: a lookup compares complete keys only.
  if (!cacheable) key.clear();
  try {
    c->lru.push_front(Entry{std::move(key), p});
  } catch (const std::bad_alloc &) {
    emoe_plan_destroy(p);
    return EMOE_ERR_OOM;
  }
  while (c->lru.size() > c->capacity) {   // least recently used plans leave
    emoe_plan_destroy(c->lru.back().plan);
    c->lru.pop_back();
    ++c->evictions;
  }
  *plan = p;
  if (hit) *hit = 0;
  return EMOE_OK;
}

emoe_status_t emoe_plan_cache_stats(emoe_plan_cache_t *c, uint64_t *hits, uint64_t *misses,
                                    uint64_t *evictions, int32_t *size) {
  if (!c) return EMOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(c->mu);
  if (hits) *hits = c->hits;
  if (misses) *misses = c->misses;
  if (evictions) *evictions = c->evictions;
  if (size) *size = (int32_t)c->lru.size();
  return EMOE_OK;
}

void emoe_plan_cache_destroy(emoe_plan_cache_t *c) {
  if (!c) return;
  for (Entry &e : c->lru) emoe_plan_destroy(e.plan);
  delete c;
}

// New block table that packs the mapped blocks into the lowest free blocks of the
// destination pool: in table order, or - given the old table - in the order of the blocks'
// old physical ids, so that a migration that walks the old pool in address order also writes
// the new pool in address order.
emoe_status_t emoe_kv_compact_table(int32_t block_tokens, int32_t n_seqs, int32_t max_blocks,
                                    const int32_t *seq_lens, int32_t nb_new, const int32_t *in_use,
                                    int32_t n_in_use, const int32_t *old_table, int32_t *table_out,
                                    int32_t *n_mapped) {
  if (block_tokens < 1 || n_seqs < 0 || max_blocks < 0 || nb_new < 0 || n_in_use < 0) return EMOE_ERR_INVALID_ARG;
  if ((n_seqs && (!seq_lens || !table_out)) || (n_in_use && !in_use)) return EMOE_ERR_INVALID_ARG;
  try {
    std::vector<char> taken((size_t)nb_new, 0);
    for (int32_t i = 0; i < n_in_use; ++i) {
      if (in_use[i] < 0 || in_use[i] >= nb_new || taken[in_use[i]]) return EMOE_ERR_BLOCK_TABLE;
      taken[in_use[i]] = 1;
    }
    // the mapped entries, as positions in the table, in the order in which they are served
    std::vector<int64_t> todo;
    for (int32_t s = 0; s < n_seqs; ++s) {
      if (seq_lens[s] < 0) return EMOE_ERR_BLOCK_TABLE;
      const int64_t n = ((int64_t)seq_lens[s] + block_tokens - 1) / block_tokens;
      if (n > max_blocks) return EMOE_ERR_BLOCK_TABLE;
      int32_t *row = table_out + (int64_t)s * max_blocks;
      for (int64_t j = 0; j < max_blocks; ++j) row[j] = -1;
      for (int64_t j = 0; j < n; ++j) {
        if (old_table && old_table[(int64_t)s * max_blocks + j] < 0) return EMOE_ERR_BLOCK_TABLE;
        todo.push_back((int64_t)s * max_blocks + j);
      }
    }
    if (old_table)
      std::stable_sort(todo.begin(), todo.end(),
                       [&](int64_t a, int64_t b) { return old_table[a] < old_table[b]; });
    int32_t next = 0;
    for (int64_t at : todo) {
      while (next < nb_new && taken[next]) ++next;
      if (next >= nb_new) {   // the pool has fewer free blocks than needed: hand out nothing
        for (int64_t k = 0; k < (int64_t)n_seqs * max_blocks; ++k) table_out[k] = -1;
        return EMOE_ERR_TOO_LARGE;
      }
      table_out[at] = next++;
    }
    if (n_mapped) *n_mapped = (int32_t)todo.size();
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}

}  // extern "C"
