// placement.cpp - a new expert placement that keeps as many experts where they are as a
// balanced placement allows.
//
// The paper wants the new placement balanced and cheap to reach (Sec. 5.2 "Expert
// Weights") but gives no algorithm.  Here: every expert is placed exactly once,
// rank sizes differ by at most one, and the number of experts that stay on a rank index
// that already holds a copy is maximal.  That is a bipartite b-matching (rank capacities,
// one unit per expert, plus a shared pool for the E mod EP ranks that take one expert
// more), solved exactly as a small max-flow; the rest is filled in id order.
#include <algorithm>
#include <cstdint>
#include <functional>
#include <new>
#include <vector>

#include "../../include/emoe.h"

extern "C" emoe_status_t emoe_place_min_transfer(int32_t n_experts, const emoe_config_t *old_cfg,
                                                 int32_t ep_new, int32_t *new_off, int32_t *new_ids,
                                                 int32_t *n_kept) {
  if (!old_cfg || !new_off || !new_ids || n_experts < 1 || ep_new < 1) return EMOE_ERR_INVALID_ARG;
  if (ep_new > EMOE_MAX_RANKS || old_cfg->ep > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  if (old_cfg->ep < 1 || !old_cfg->place_off || !old_cfg->place_ids || old_cfg->place_off[0] != 0)
    return EMOE_ERR_PLACEMENT;
  try {
    const int E = n_experts, R = ep_new, Rk = std::min<int>(R, old_cfg->ep);
    // holds[r]: experts old rank r has (ranks that exist on both sides only)
    std::vector<std::vector<int>> holds(Rk);
    std::vector<char> seen(E, 0);
    for (int r = 0; r < old_cfg->ep; ++r) {
      if (old_cfg->place_off[r + 1] < old_cfg->place_off[r]) return EMOE_ERR_PLACEMENT;
      for (int i = old_cfg->place_off[r]; i < old_cfg->place_off[r + 1]; ++i) {
        const int e = old_cfg->place_ids[i];
        if (e < 0 || e >= E) return EMOE_ERR_PLACEMENT;
        seen[e] = 1;
        if (r < Rk && std::find(holds[r].begin(), holds[r].end(), e) == holds[r].end()) holds[r].push_back(e);
      }
    }
    for (int e = 0; e < E; ++e)
      if (!seen[e]) return EMOE_ERR_PLACEMENT;  // an expert nobody holds cannot be placed

    const int base = E / R, extra = E % R;
    // Max flow: S -> rank (base), S -> pool (extra), pool -> rank (1), rank -> expert it
    // holds (1), expert -> T (1).  A unit of flow = an expert that stays on that rank.
    struct Edge { int to, cap; };
    std::vector<Edge> edges;
    const int S = 0, T = 1, POOL = 2, RANK0 = 3, EXP0 = 3 + Rk, N = 3 + Rk + E;
    std::vector<std::vector<int>> adj(N);
    auto add = [&](int u, int v, int c) {
      adj[u].push_back((int)edges.size()); edges.push_back({v, c});
      adj[v].push_back((int)edges.size()); edges.push_back({u, 0});
    };
    add(S, POOL, extra);
    std::vector<int> pool_edge(Rk, -1);
    for (int r = 0; r < Rk; ++r) {
      add(S, RANK0 + r, base);
      pool_edge[r] = (int)edges.size();
      add(POOL, RANK0 + r, 1);
      for (int e : holds[r]) add(RANK0 + r, EXP0 + e, 1);
    }
    for (int e = 0; e < E; ++e) add(EXP0 + e, T, 1);
    std::vector<char> visited(N);
    std::function<bool(int)> push = [&](int u) -> bool {  // one augmenting path by depth-first search
      if (u == T) return true;
      visited[u] = 1;
      for (int id : adj[u]) {
        Edge &ed = edges[id];
        if (ed.cap <= 0 || visited[ed.to]) continue;
        if (push(ed.to)) { ed.cap--; edges[id ^ 1].cap++; return true; }
      }
      return false;
    };
    for (;;) {
      std::fill(visited.begin(), visited.end(), 0);
      if (!push(S)) break;
    }
    std::vector<int> kept_by(E, -1);
    std::vector<char> has_extra(Rk, 0);
    int extra_used = 0;
    for (int r = 0; r < Rk; ++r) {
      if (edges[pool_edge[r]].cap == 0) { has_extra[r] = 1; ++extra_used; }
      for (int id : adj[RANK0 + r]) {
        const Edge &ed = edges[id];
        if ((id & 1) == 0 && ed.to >= EXP0 && ed.cap == 0) kept_by[ed.to - EXP0] = r;
      }
    }
    // final capacities: leftover extra slots go to the lowest ranks without one
    std::vector<int> cap(R, base);
    for (int r = 0; r < Rk; ++r)
      if (has_extra[r]) cap[r]++;
    int left = extra - extra_used;
    for (int r = 0; r < R && left > 0; ++r) {
      const bool had = r < Rk && has_extra[r];
      if (!had) { cap[r]++; --left; }
    }
    std::vector<std::vector<int>> out(R);
    int kept = 0;
    for (int e = 0; e < E; ++e)
      if (kept_by[e] >= 0) { out[kept_by[e]].push_back(e); ++kept; }
    int r = 0;
    for (int e = 0; e < E; ++e) {
      if (kept_by[e] >= 0) continue;
      while (r < R && (int)out[r].size() >= cap[r]) ++r;
      if (r >= R) return EMOE_ERR_PLACEMENT;  // not reached: capacities sum to E
      out[r].push_back(e);
    }
    new_off[0] = 0;
    int k = 0;
    for (int q = 0; q < R; ++q) {
      std::sort(out[q].begin(), out[q].end());
      for (int e : out[q]) new_ids[k++] = e;
      new_off[q + 1] = k;
    }
    if (n_kept) *n_kept = kept;
  } catch (const std::bad_alloc &) {
    return EMOE_ERR_OOM;
  }
  return EMOE_OK;
}
