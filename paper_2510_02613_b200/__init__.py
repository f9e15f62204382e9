"""B200-native re-layout of MoE weights and paged KV cache for an elastic scaling
step (expert re-pack for EP a->b, attention re-slice and KV head re-split for TP
c->d).  The work is done by libemoe.so (host planner, C ABI, sm_100a copy
kernels); this package is its thin ctypes binding."""
from .binding import (EXPORTS, MAX_RANKS, PHASE_ATTN, PHASE_EXPERTS, PHASE_KV, PHASE_STEP, PLAN_HOST_ONLY, PLAN_HOST_STEP,
                      SEGMENT_DTYPE, SIDE_NEW, SIDE_OLD, EmoeError, InplacePlan, Plan, PlanCache, VmmPool, VmmSlots, kv_compact_table, segments_validate, lib, library_path,
                      strerror, vmm_dry_run, ipc_export, ipc_open, ipc_close,
                      place_min_transfer)

__all__ = ["EXPORTS", "MAX_RANKS", "PHASE_ATTN", "PHASE_EXPERTS", "PHASE_KV", "PHASE_STEP", "PLAN_HOST_ONLY", "PLAN_HOST_STEP",
           "SEGMENT_DTYPE", "SIDE_NEW", "SIDE_OLD", "EmoeError", "InplacePlan", "Plan", "PlanCache", "kv_compact_table", "segments_validate", "VmmPool", "VmmSlots", "lib", "library_path",
           "strerror", "vmm_dry_run", "ipc_export", "ipc_open", "ipc_close", "place_min_transfer"]
