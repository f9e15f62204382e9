// validate.cpp - host-side self-check of a copy plan: the race and bounds check of this
// library.  Copy kernels race only if two of them write the same byte, and fault only if a run
// leaves its arena; both are properties of the segment list and can be checked before anything
// is launched: every source run inside its arena, every destination run inside its arena,
// destination runs pairwise disjoint, and - where the phase must fill its arenas - the
// destination runs tiling them exactly.
#include <algorithm>
#include <cstdint>
#include <new>
#include <utility>
#include <vector>

#include "planner.h"

using namespace emoe;

extern "C" {

emoe_status_t emoe_segments_validate(const emoe_segment_t *segs, uint64_t n_segs, const uint64_t *arena_old,
                                     int32_t n_old, const uint64_t *arena_new, int32_t n_new,
                                     int32_t must_tile, uint64_t *bad_segment) {
  if ((n_segs && !segs) || n_old < 0 || n_new < 0 || (n_old && !arena_old) || (n_new && !arena_new))
    return EMOE_ERR_INVALID_ARG;
  auto fail = [&](uint64_t i) {
    if (bad_segment) *bad_segment = i;
    return EMOE_ERR_PLAN_CHECK;
  };
  try {
    // (start, end, segment) of every destination run, per new rank
    std::vector<std::vector<std::pair<std::pair<uint64_t, uint64_t>, uint64_t>>> runs((size_t)n_new);
    for (uint64_t i = 0; i < n_segs; ++i) {
      const emoe_segment_t &s = segs[i];
      if (s.src_rank >= (uint32_t)n_old || s.dst_rank >= (uint32_t)n_new) return fail(i);
      if (s.n_runs == 0 || s.run_bytes == 0) continue;
      const uint64_t last = (uint64_t)(s.n_runs - 1);
      // bounds, written so that nothing overflows: off + last * pitch + run <= arena
      auto inside = [&](uint64_t off, uint64_t pitch, uint64_t arena) {
        if (s.run_bytes > arena || off > arena - s.run_bytes) return false;
        if (last == 0) return true;
        return pitch <= (arena - s.run_bytes - off) / last;
      };
      if (!inside(s.src_off, s.src_pitch, arena_old[s.src_rank])) return fail(i);
      if (!inside(s.dst_off, s.dst_pitch, arena_new[s.dst_rank])) return fail(i);
      if (last > 0 && s.dst_pitch < s.run_bytes) return fail(i);   // a segment's own runs overlap
      auto &mine = runs[s.dst_rank];
      if (last == 0 || s.dst_pitch == s.run_bytes) {
        mine.push_back({{s.dst_off, s.dst_off + (last + 1) * s.run_bytes}, i});
      } else {
        for (uint64_t r = 0; r <= last; ++r)
          mine.push_back({{s.dst_off + r * s.dst_pitch, s.dst_off + r * s.dst_pitch + s.run_bytes}, i});
      }
    }
    for (int32_t rk = 0; rk < n_new; ++rk) {
      auto &mine = runs[(size_t)rk];
      std::sort(mine.begin(), mine.end());
      uint64_t end = 0;
      for (const auto &iv : mine) {
        if (iv.first.first < end) return fail(iv.second);                    // two writers of one byte
        if (must_tile && iv.first.first != end) return fail(iv.second);      // a byte nobody writes
        end = iv.first.second;
      }
      if (must_tile && end != arena_new[rk]) return fail(mine.empty() ? n_segs : mine.back().second);
    }
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}

}  // extern "C"
