/* A C99 caller of the library: proves that include/emoe.h is plain C and that a host-only
 * plan can be made, queried and destroyed without any CUDA device. */
#include <stdio.h>
#include <string.h>

#include "emoe.h"

int main(void) {
  emoe_shape_t sh = {2, 4, 0, 64, 32, 4, 4, 16, 4, 2};
  int32_t old_off[3] = {0, 2, 4}, old_ids[4] = {0, 1, 2, 3};
  int32_t new_off[5] = {0, 1, 2, 3, 4}, new_ids[4] = {0, 1, 2, 3};
  int32_t seq_lens[1] = {7}, bt_old[2] = {1, 0}, bt_new[2] = {2, 1};
  emoe_config_t oc = {2, 1, old_off, old_ids, 2, 1, 2, seq_lens, bt_old};
  emoe_config_t nc = {4, 2, new_off, new_ids, 3, 1, 2, seq_lens, bt_new};
  emoe_plan_t *plan = NULL;
  emoe_status_t st = emoe_plan_create(&sh, &oc, &nc, EMOE_PLAN_HOST_ONLY, &plan);
  if (st != EMOE_OK) { printf("create: %s\n", emoe_strerror(st)); return 1; }
  uint64_t moved = 0, read = 0, nseg = 0, bytes = 0;
  int32_t n = 0;
  if (emoe_plan_stats(plan, EMOE_PHASE_EXPERTS, &moved, &read, &nseg) != EMOE_OK) return 2;
  if (moved != 2ull * 3 * 4 * 64 * 32 * 2) return 3;            /* L * 3 * experts * m */
  if (emoe_plan_num_ranks(plan, EMOE_PHASE_KV, EMOE_SIDE_NEW, &n) != EMOE_OK || n != 2) return 4;
  if (emoe_plan_arena_bytes(plan, EMOE_PHASE_KV, EMOE_SIDE_NEW, 1, &bytes) != EMOE_OK) return 5;
  if (bytes != 2ull * 2 * 3 * 4 * 2 * 16 * 2) return 6;         /* L * 2 * NB * B * heads * hd * b */
  /* a host-only plan must refuse to run, and bad input must map to its code */
  {
    const void *src[2] = {(void *)16, (void *)32};
    void *dst[4] = {(void *)48, (void *)64, (void *)80, (void *)96};
    if (emoe_reshard_experts(plan, src, dst, NULL) != EMOE_ERR_CUDA) return 7;
  }
  emoe_plan_destroy(plan);
  nc.tp = 3;                                                    /* 3 does not divide 4 heads */
  if (emoe_plan_create(&sh, &oc, &nc, EMOE_PLAN_HOST_ONLY, &plan) != EMOE_ERR_SHAPE) return 8;
  if (strcmp(emoe_strerror(EMOE_OK), "ok") != 0) return 9;
  nc.tp = 2;
  {
    /* scale tensors in the same plan: weights, then (256-byte aligned) 8 bytes per matrix */
    emoe_plan_options_t opt;
    memset(&opt, 0, sizeof(opt));
    opt.expert_scale_bytes = 8;
    if (emoe_plan_create_ex(&sh, &oc, &nc, EMOE_PLAN_HOST_ONLY, &opt, &plan) != EMOE_OK) return 10;
    if (emoe_plan_arena_bytes(plan, EMOE_PHASE_EXPERTS, EMOE_SIDE_NEW, 0, &bytes) != EMOE_OK) return 11;
    if (bytes != 2ull * 3 * 1 * 64 * 32 * 2 + 2ull * 3 * 1 * 8) return 12;   /* 24576 is a multiple of 256 */
    emoe_plan_destroy(plan);
  }
  {
    /* in-place expert step: device 0 [0, 1, free], device 1 [2, 3, free] -> 0 wants {0, 2}, 1 wants {3, 1} */
    int32_t slot_off[3] = {0, 3, 6}, slot_ids[6] = {0, 1, -1, 2, 3, -1};
    int32_t cap[2] = {3, 3}, want_off[3] = {0, 2, 4}, want[4] = {0, 2, 3, 1}, table[3], n_slots = 0;
    if (emoe_plan_create_inplace(&sh, 2, slot_off, slot_ids, 2, cap, want_off, want, EMOE_PLAN_HOST_ONLY,
                                 &plan) != EMOE_OK) return 13;
    if (emoe_plan_slot_table(plan, 0, table, 3, &n_slots) != EMOE_OK || n_slots != 3) return 14;
    if (table[0] != 0 || table[1] != -1 || table[2] != 2) return 15;
    if (emoe_plan_stats(plan, EMOE_PHASE_EXPERTS, &moved, &read, &nseg) != EMOE_OK) return 16;
    if (moved != 2ull * 2 * 3 * 64 * 32 * 2) return 17;         /* two arrivals only */
    emoe_plan_destroy(plan);
  }
  {
    /* plan cache and the compacting block table */
    emoe_plan_cache_t *cache = NULL;
    int32_t hit = -1, bt[2] = {9, 9}, mapped = 0, in_use[1] = {0};
    uint64_t hits = 0, misses = 0;
    if (emoe_plan_cache_create(2, &cache) != EMOE_OK) return 18;
    if (emoe_plan_cache_get(cache, &sh, &oc, &nc, EMOE_PLAN_HOST_ONLY, NULL, &plan, &hit) != EMOE_OK || hit) return 19;
    if (emoe_plan_cache_get(cache, &sh, &oc, &nc, EMOE_PLAN_HOST_ONLY, NULL, &plan, &hit) != EMOE_OK || !hit) return 20;
    if (emoe_plan_cache_stats(cache, &hits, &misses, NULL, NULL) != EMOE_OK || hits != 1 || misses != 1) return 21;
    emoe_plan_cache_destroy(cache);
    if (emoe_kv_compact_table(4, 1, 2, seq_lens, 3, in_use, 1, NULL, bt, &mapped) != EMOE_OK) return 22;
    if (bt[0] != 1 || bt[1] != 2 || mapped != 2) return 23;
  }
  printf("c abi ok\n");
  return 0;
}
