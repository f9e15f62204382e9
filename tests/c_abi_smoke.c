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
  printf("c abi ok\n");
  return 0;
}
