// planner.cpp - host planner: validation, move enumeration, coalescing.
#include "planner.h"

#include <algorithm>
#include <map>
#include <utility>

namespace emoe {
namespace {

uint32_t pow2_align(uint64_t v) {  // largest power of two <= 16 dividing v (16 for v == 0)
  uint32_t a = 16;
  while (a > 1 && (v % a) != 0) a >>= 1;
  return a;
}

void finish_segment(PhasePlan *pp, Segment s, const std::vector<Dst> &dsts) {
  // a strided segment whose pitches equal the run size on both sides is contiguous
  bool dense = s.n_runs > 1 && s.src_pitch == s.run_bytes;
  for (const Dst &d : dsts) dense = dense && d.pitch == s.run_bytes;
  if (dense) {
    s.run_bytes *= s.n_runs;
    s.n_runs = 1;
  }
  uint32_t a = std::min(pow2_align(s.src_off), pow2_align(s.run_bytes));
  if (s.n_runs > 1) a = std::min(a, pow2_align(s.src_pitch));
  for (const Dst &d : dsts) {
    a = std::min(a, pow2_align(d.off));
    if (s.n_runs > 1) a = std::min(a, pow2_align(d.pitch));
  }
  s.align = a;
  s.n_dst = (uint32_t)dsts.size();
  s.dst_first = (uint32_t)pp->dsts.size();
  s.pad = 0;
  pp->dsts.insert(pp->dsts.end(), dsts.begin(), dsts.end());
  pp->segs.push_back(s);
  pp->bytes_read += (uint64_t)s.n_runs * s.run_bytes;
  pp->bytes_moved += (uint64_t)s.n_runs * s.run_bytes * dsts.size();
}

struct Placement {
  int ep = 0;
  std::vector<std::vector<int32_t>> ids;
};

emoe_status_t read_placement(const emoe_config_t &cfg, int n_experts, Placement *out) {
  if (cfg.ep < 1 || cfg.tp < 1) return EMOE_ERR_INVALID_ARG;
  if (cfg.ep > EMOE_MAX_RANKS || cfg.tp > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  if (!cfg.place_off || !cfg.place_ids) return EMOE_ERR_INVALID_ARG;
  if (cfg.place_off[0] != 0) return EMOE_ERR_PLACEMENT;
  out->ep = cfg.ep;
  out->ids.assign(cfg.ep, {});
  std::vector<int> seen_total(n_experts, 0);
  for (int r = 0; r < cfg.ep; ++r) {
    if (cfg.place_off[r + 1] < cfg.place_off[r]) return EMOE_ERR_PLACEMENT;
    std::vector<char> seen(n_experts, 0);
    for (int i = cfg.place_off[r]; i < cfg.place_off[r + 1]; ++i) {
      const int32_t e = cfg.place_ids[i];
      if (e < 0 || e >= n_experts) return EMOE_ERR_PLACEMENT;
      if (seen[e]) return EMOE_ERR_PLACEMENT;  // the same expert twice on one rank
      seen[e] = 1;
      seen_total[e]++;
      out->ids[r].push_back(e);
    }
  }
  for (int e = 0; e < n_experts; ++e)
    if (!seen_total[e]) return EMOE_ERR_PLACEMENT;  // an expert nobody holds would be lost
  return EMOE_OK;
}

emoe_status_t read_block_pairs(const emoe_shape_t &sh, const emoe_config_t &o,
                               const emoe_config_t &n, std::vector<uint32_t> *po,
                               std::vector<uint32_t> *pn) {
  if (o.n_seqs != n.n_seqs || o.n_seqs < 0) return EMOE_ERR_BLOCK_TABLE;
  if (o.kv_num_blocks < 0 || n.kv_num_blocks < 0) return EMOE_ERR_BLOCK_TABLE;
  if (o.n_seqs == 0) return EMOE_OK;
  if (!o.seq_lens || !n.seq_lens || !o.block_table || !n.block_table) return EMOE_ERR_INVALID_ARG;
  std::vector<char> used_o(o.kv_num_blocks, 0), used_n(n.kv_num_blocks, 0);
  const int64_t B = sh.kv_block_tokens;
  for (int s = 0; s < o.n_seqs; ++s) {
    if (o.seq_lens[s] != n.seq_lens[s] || o.seq_lens[s] < 0) return EMOE_ERR_BLOCK_TABLE;
    const int64_t nblk = (o.seq_lens[s] + B - 1) / B;
    if (nblk > o.max_blocks || nblk > n.max_blocks) return EMOE_ERR_BLOCK_TABLE;
    for (int64_t j = 0; j < nblk; ++j) {
      const int32_t a = o.block_table[(int64_t)s * o.max_blocks + j];
      const int32_t b = n.block_table[(int64_t)s * n.max_blocks + j];
      if (a < 0 || a >= o.kv_num_blocks || b < 0 || b >= n.kv_num_blocks)
        return EMOE_ERR_BLOCK_TABLE;
      if (used_o[a] || used_n[b]) return EMOE_ERR_BLOCK_TABLE;  // shared blocks unsupported
      used_o[a] = used_n[b] = 1;
      po->push_back((uint32_t)a);
      pn->push_back((uint32_t)b);
    }
  }
  return EMOE_OK;
}

// ---- experts ----------------------------------------------------------------------------

struct ExpertMove { int rs, ss, rd, sd; };

// Moves -> segments.  slots_old / slots_new: slots per arena (the slot stride of a layer slab).
// Single-destination sources: runs of consecutive slots on both sides merge (dense layout
// only); a source with several destinations becomes one segment that is read once.
// m: bytes of the tensor that moves per (layer, projection, slot) - the expert matrix, or the
// scale tensor that goes with it; base_old / base_new: where that tensor's [L][3][n] array
// starts inside each arena (null: at 0).
void emit_expert_moves(const emoe_shape_t &sh, const std::vector<uint64_t> &slots_old,
                       const std::vector<uint64_t> &slots_new, uint64_t slab, uint64_t m,
                       const std::vector<uint64_t> *base_old, const std::vector<uint64_t> *base_new,
                       const std::vector<ExpertMove> &moves, std::map<std::pair<int, int>, int> &fan,
                       bool fused_w13, PhasePlan *pp) {
  const uint32_t runs = (uint32_t)sh.n_layers * 3;
  const size_t seg0 = pp->segs.size();
  // single-destination sources: merge runs of consecutive slots on both sides (dense layout only)
  std::map<std::pair<int, int>, std::vector<Dst>> multi;
  size_t i = 0;
  while (i < moves.size()) {
    const ExpertMove &a = moves[i];
    const uint64_t n_old = slots_old[a.rs], n_new = slots_new[a.rd];
    if (fan[{a.rs, a.ss}] > 1) {
      // fused layout: off = slot index, pitch = slot count; resolved to bytes below
      if (fused_w13) multi[{a.rs, a.ss}].push_back({(uint64_t)a.sd, n_new, (uint32_t)a.rd, 0});
      else multi[{a.rs, a.ss}].push_back({(uint64_t)a.sd * slab, n_new * slab, (uint32_t)a.rd, 0});
      ++i;
      continue;
    }
    size_t j = i + 1;
    while (slab == m && j < moves.size() && moves[j].rd == a.rd && moves[j].rs == a.rs &&
           moves[j].sd == moves[j - 1].sd + 1 && moves[j].ss == moves[j - 1].ss + 1 &&
           fan[{moves[j].rs, moves[j].ss}] == 1)
      ++j;
    Segment s{};
    s.src_rank = (uint32_t)a.rs;
    if (!fused_w13) {
      s.src_off = (uint64_t)a.ss * slab;
      s.run_bytes = (uint64_t)(j - i) * m;
      s.src_pitch = n_old * slab;
      s.n_runs = runs;
      finish_segment(pp, s, {Dst{(uint64_t)a.sd * slab, n_new * slab, (uint32_t)a.rd, 0}});
    } else {  // per layer: the slots' gate|up pairs, then their down matrices
      s.n_runs = (uint32_t)sh.n_layers;
      s.src_pitch = 3 * n_old * m;
      s.src_off = (uint64_t)a.ss * 2 * m;
      s.run_bytes = (uint64_t)(j - i) * 2 * m;
      finish_segment(pp, s, {Dst{(uint64_t)a.sd * 2 * m, 3 * n_new * m, (uint32_t)a.rd, 0}});
      s.src_off = n_old * 2 * m + (uint64_t)a.ss * m;
      s.run_bytes = (uint64_t)(j - i) * m;
      finish_segment(pp, s, {Dst{n_new * 2 * m + (uint64_t)a.sd * m, 3 * n_new * m, (uint32_t)a.rd, 0}});
    }
    i = j;
  }
  // replicated sources: read once, write to every destination
  for (const auto &kv : multi) {
    Segment s{};
    s.src_rank = (uint32_t)kv.first.first;
    const uint64_t n_old = slots_old[kv.first.first], ss = (uint64_t)kv.first.second;
    if (!fused_w13) {
      s.src_off = ss * slab;
      s.run_bytes = m;
      s.src_pitch = n_old * slab;
      s.n_runs = runs;
      finish_segment(pp, s, kv.second);
    } else {
      std::vector<Dst> d13, d2;
      for (const Dst &d : kv.second) {  // d.off = slot, d.pitch = slots of that rank
        d13.push_back({d.off * 2 * m, 3 * d.pitch * m, d.rank, 0});
        d2.push_back({d.pitch * 2 * m + d.off * m, 3 * d.pitch * m, d.rank, 0});
      }
      s.n_runs = (uint32_t)sh.n_layers;
      s.src_pitch = 3 * n_old * m;
      s.src_off = ss * 2 * m;
      s.run_bytes = 2 * m;
      finish_segment(pp, s, d13);
      s.src_off = n_old * 2 * m + ss * m;
      s.run_bytes = m;
      finish_segment(pp, s, d2);
    }
  }
  // the tensor's array does not start at the arena's first byte: shift what was just emitted
  if (base_old || base_new)
    for (size_t k = seg0; k < pp->segs.size(); ++k) {
      Segment &sg = pp->segs[k];
      if (base_old) sg.src_off += (*base_old)[sg.src_rank];
      for (uint32_t j = 0; j < sg.n_dst; ++j) {
        Dst &dd = pp->dsts[sg.dst_first + j];
        if (base_new) dd.off += (*base_new)[dd.rank];
      }
    }
}


// slab: distance between consecutive slots of an arena (= m for the dense layout; the
// paged store pads every matrix to its allocation granularity).  remaps: if non-null,
// a destination slot whose source sits on the same rank index is recorded there instead
// of being copied (that device already holds the bytes).
// fused_w13 (dense layout only): per layer a [n][gate|up] tensor, then the [n][down] one.
// scale_bytes > 0: every matrix travels with a scale tensor of that many bytes; an arena is
// then the weight array [L][3][n][m], and from the next multiple of 256 bytes on the scale
// array [L][3][n][scale_bytes].
void plan_experts(const emoe_shape_t &sh, const Placement &po, const Placement &pn, uint64_t slab,
                  std::vector<Remap> *remaps, bool fused_w13, uint64_t scale_bytes, PhasePlan *pp) {
  const uint64_t m = (uint64_t)sh.d_model * sh.d_ff * sh.elem_bytes;
  const uint32_t runs = (uint32_t)sh.n_layers * 3;
  const int n_experts = sh.n_routed + sh.n_shared;
  std::vector<uint64_t> scale_base_old, scale_base_new;
  auto arena = [&](uint64_t n, std::vector<uint64_t> *bases) {
    const uint64_t w = runs * n * slab;
    if (!scale_bytes) return w;
    bases->push_back((w + 255) / 256 * 256);
    return bases->back() + runs * n * scale_bytes;
  };
  for (int r = 0; r < po.ep; ++r) pp->arena_old.push_back(arena(po.ids[r].size(), &scale_base_old));
  for (int r = 0; r < pn.ep; ++r) pp->arena_new.push_back(arena(pn.ids[r].size(), &scale_base_new));

  // every old copy of every expert, in (rank, slot) order
  std::vector<std::vector<std::pair<int, int>>> copies(n_experts);
  for (int r = 0; r < po.ep; ++r)
    for (int s = 0; s < (int)po.ids[r].size(); ++s) copies[po.ids[r][s]].push_back({r, s});

  // source of every destination slot: the copy on the same rank index, else the first
  std::vector<ExpertMove> moves;
  std::vector<uint64_t> slots_old, slots_new;
  for (int r = 0; r < po.ep; ++r) slots_old.push_back(po.ids[r].size());
  for (int r = 0; r < pn.ep; ++r) slots_new.push_back(pn.ids[r].size());
  std::map<std::pair<int, int>, int> fan;  // (src rank, src slot) -> number of destinations
  for (int rd = 0; rd < pn.ep; ++rd)
    for (int sd = 0; sd < (int)pn.ids[rd].size(); ++sd) {
      const auto &c = copies[pn.ids[rd][sd]];
      std::pair<int, int> src = c.front();
      for (const auto &x : c)
        if (x.first == rd) { src = x; break; }
      if (remaps && src.first == rd) {
        remaps->push_back({(uint32_t)src.first, (uint32_t)src.second, (uint32_t)rd, (uint32_t)sd});
        continue;
      }
      moves.push_back({src.first, src.second, rd, sd});
      fan[src]++;
    }

  emit_expert_moves(sh, slots_old, slots_new, slab, m, nullptr, nullptr, moves, fan, fused_w13, pp);
  if (scale_bytes)   // the same moves once more for the scale tensors (plain [L][3][n] array)
    emit_expert_moves(sh, slots_old, slots_new, scale_bytes, scale_bytes, &scale_base_old, &scale_base_new,
                      moves, fan, false, pp);
}

// ---- attention --------------------------------------------------------------------------

// q, k and v rows of the fused-qkv arena: one move per head (a head's hd rows are contiguous
// on both sides), moves that are neighbours on both sides merged, one strided segment
// (a run per layer) per merged move.  Row groups: for every KV head of a rank, the rank's
// query heads of that group, then the k head, then the v head.
void plan_fused_qkv(const emoe_shape_t &sh, int c, int d, uint64_t layer_c, uint64_t layer_d,
                    PhasePlan *pp) {
  const uint64_t head = (uint64_t)sh.head_dim * sh.d_model * sh.elem_bytes;
  const uint32_t hq = sh.n_q_heads, hkv = sh.n_kv_heads;
  auto kvh = [&](int T) { return (uint64_t)kv_heads_per_rank(hkv, T); };
  auto qpg = [&](int T) { return (uint64_t)(hq / T) / kvh(T); };
  auto q_off = [&](int T, uint64_t h) {
    const uint64_t local = h % (hq / T), j = local / qpg(T), i = local % qpg(T);
    return (j * (qpg(T) + 2) + i) * head;
  };
  auto kv_off = [&](int T, uint64_t j, int which) { return (j * (qpg(T) + 2) + qpg(T) + which) * head; };
  struct Mv { uint32_t ro, rn; uint64_t so, dn, bytes; };
  std::vector<Mv> mv;
  for (uint32_t h = 0; h < hq; ++h)
    mv.push_back({h / (hq / c), h / (hq / d), q_off(c, h), q_off(d, h), head});
  for (int which = 0; which < 2; ++which)
    for (int rn = 0; rn < d; ++rn)
      for (uint32_t jn = 0; jn < kvh(d); ++jn) {
        const uint32_t g = kv_first_head(hkv, d, rn) + jn;
        const uint32_t ro = kv_source_rank(hkv, c, g, rn);
        mv.push_back({ro, (uint32_t)rn, kv_off(c, g - kv_first_head(hkv, c, ro), which),
                      kv_off(d, jn, which), head});
      }
  std::sort(mv.begin(), mv.end(), [](const Mv &a, const Mv &b) {
    return a.rn != b.rn ? a.rn < b.rn : a.dn < b.dn;
  });
  size_t i = 0;
  while (i < mv.size()) {
    Mv a = mv[i];
    size_t j = i + 1;
    while (j < mv.size() && mv[j].rn == a.rn && mv[j].ro == a.ro && mv[j].dn == a.dn + a.bytes &&
           mv[j].so == a.so + a.bytes) {
      a.bytes += mv[j].bytes;
      ++j;
    }
    Segment s{};
    s.src_off = a.so;
    s.run_bytes = a.bytes;
    s.src_pitch = layer_c;
    s.n_runs = (uint32_t)sh.n_layers;
    s.src_rank = a.ro;
    finish_segment(pp, s, {Dst{a.dn, layer_d, a.rn, 0}});
    i = j;
  }
}

void plan_attn(const emoe_shape_t &sh, int c, int d, bool fused_qkv, PhasePlan *pp) {
  const uint64_t D = sh.d_model, b = sh.elem_bytes, hd = sh.head_dim;
  const uint64_t row = D * b;
  const uint32_t hkv = sh.n_kv_heads;
  auto q_bytes = [&](int T) { return (uint64_t)(sh.n_q_heads / T) * hd * row; };
  auto kv_bytes = [&](int T) { return (uint64_t)kv_heads_per_rank(hkv, T) * hd * row; };
  auto layer_bytes = [&](int T) { return 2 * q_bytes(T) + 2 * kv_bytes(T); };
  const uint32_t L = sh.n_layers;
  pp->arena_old.assign(c, L * layer_bytes(c));
  pp->arena_new.assign(d, L * layer_bytes(d));

  if (c == d) {  // fixed TP: every shard carries over whole (provisioning a new replica)
    for (int t = 0; t < c; ++t) {
      Segment s{};
      s.run_bytes = L * layer_bytes(c);
      s.n_runs = 1;
      s.src_pitch = s.run_bytes;
      s.src_rank = (uint32_t)t;
      finish_segment(pp, s, {Dst{0, s.run_bytes, (uint32_t)t, 0}});
    }
    return;
  }
  if (fused_qkv) plan_fused_qkv(sh, c, d, layer_bytes(c), layer_bytes(d), pp);
  // q: intersect old and new row ranges of the logical matrix
  if (!fused_qkv) {
    const uint64_t rows = (uint64_t)sh.n_q_heads * hd;
    const uint64_t rc = rows / c, rd = rows / d;
    for (int ro = 0; ro < c; ++ro)
      for (int rn = 0; rn < d; ++rn) {
        const uint64_t lo = std::max(ro * rc, rn * rd), hi = std::min((ro + 1) * rc, (rn + 1) * rd);
        if (lo >= hi) continue;
        Segment s{};
        s.src_off = (lo - ro * rc) * row;
        s.run_bytes = (hi - lo) * row;
        s.src_pitch = layer_bytes(c);
        s.n_runs = L;
        s.src_rank = (uint32_t)ro;
        finish_segment(pp, s, {Dst{(lo - rn * rd) * row, layer_bytes(d), (uint32_t)rn, 0}});
      }
  }
  // k, v: every new rank's heads, grouped into runs of heads that are consecutive on one
  // old rank (with more ranks than KV heads a head has several holders: see kv_source_rank)
  for (int t = 1; t < 3 && !fused_qkv; ++t) {
    auto piece = [&](int T) { return t == 1 ? q_bytes(T) : q_bytes(T) + kv_bytes(T); };
    const uint32_t hn = kv_heads_per_rank(hkv, d);
    for (int rn = 0; rn < d; ++rn) {
      uint32_t hl = 0;
      while (hl < hn) {
        const uint32_t g0 = kv_first_head(hkv, d, rn) + hl;
        const uint32_t ro = kv_source_rank(hkv, c, g0, rn);
        uint32_t n = 1;
        while (hl + n < hn && kv_source_rank(hkv, c, g0 + n, rn) == ro) ++n;
        Segment s{};
        s.src_off = piece(c) + (uint64_t)(g0 - kv_first_head(hkv, c, ro)) * hd * row;
        s.run_bytes = (uint64_t)n * hd * row;
        s.src_pitch = layer_bytes(c);
        s.n_runs = L;
        s.src_rank = ro;
        finish_segment(pp, s, {Dst{piece(d) + (uint64_t)hl * hd * row, layer_bytes(d), (uint32_t)rn, 0}});
        hl += n;
      }
    }
  }
  // o: intersect old and new column ranges; one strided segment per (layer, overlap)
  const uint64_t cols = (uint64_t)sh.n_q_heads * hd, cc = cols / c, cd = cols / d;
  const uint64_t o_c = q_bytes(c) + 2 * kv_bytes(c), o_d = q_bytes(d) + 2 * kv_bytes(d);
  for (uint32_t l = 0; l < L; ++l)
    for (int ro = 0; ro < c; ++ro)
      for (int rn = 0; rn < d; ++rn) {
        const uint64_t lo = std::max(ro * cc, rn * cd), hi = std::min((ro + 1) * cc, (rn + 1) * cd);
        if (lo >= hi) continue;
        Segment s{};
        s.src_off = l * layer_bytes(c) + o_c + (lo - ro * cc) * b;
        s.run_bytes = (hi - lo) * b;
        s.src_pitch = cc * b;
        s.n_runs = (uint32_t)D;
        s.src_rank = (uint32_t)ro;
        finish_segment(pp, s,
                       {Dst{l * layer_bytes(d) + o_d + (lo - rn * cd) * b, cd * b, (uint32_t)rn, 0}});
      }
}

// ---- KV ---------------------------------------------------------------------------------

void plan_kv(const emoe_shape_t &sh, const emoe_config_t &o, const emoe_config_t &n,
             std::vector<uint32_t> pair_old, std::vector<uint32_t> pair_new, bool head_major,
             HostPlan *hp) {
  PhasePlan *pp = &hp->phase[EMOE_PHASE_KV];
  KvPlan &kv = hp->kv;
  const uint64_t vec = (uint64_t)sh.head_dim * sh.elem_bytes, B = sh.kv_block_tokens;
  const uint64_t L = sh.n_layers;
  kv.c = o.tp; kv.d = n.tp;
  kv.n_layers = sh.n_layers; kv.block_tokens = sh.kv_block_tokens; kv.hkv = sh.n_kv_heads;
  kv.head_bytes = vec; kv.nb_old = o.kv_num_blocks; kv.nb_new = n.kv_num_blocks;
  kv.head_split_changes = (o.tp != n.tp);
  kv.hc = kv_heads_per_rank(kv.hkv, kv.c);
  kv.hn = kv_heads_per_rank(kv.hkv, kv.d);
  kv.replicated = kv.c > kv.hkv || kv.d > kv.hkv;
  kv.src_rank.clear();
  kv.src_head.clear();
  std::vector<char> read_slot((size_t)kv.c * kv.hc, 0);
  for (uint32_t rn = 0; rn < kv.d; ++rn)
    for (uint32_t hl = 0; hl < kv.hn; ++hl) {
      const uint32_t g = kv_first_head(kv.hkv, kv.d, rn) + hl;
      const uint32_t ro = kv_source_rank(kv.hkv, kv.c, g, rn);
      const uint32_t ho = g - kv_first_head(kv.hkv, kv.c, ro);
      kv.src_rank.push_back((uint8_t)ro);
      kv.src_head.push_back((uint16_t)ho);
      read_slot[(size_t)ro * kv.hc + ho] = 1;
    }
  uint64_t heads_read = 0;
  for (char x : read_slot) heads_read += x;
  const uint64_t blk_old = B * kv.hc * vec, blk_new = B * kv.hn * vec;
  pp->arena_old.assign(o.tp, L * 2 * o.kv_num_blocks * blk_old);
  pp->arena_new.assign(n.tp, L * 2 * n.kv_num_blocks * blk_new);
  const uint64_t n_pairs = pair_old.size();
  const uint64_t per_head = L * 2 * n_pairs * B * vec;

  kv.pair_old = pair_old;  // kept in both cases: the fixed-scratch entry point reads them
  kv.pair_new = pair_new;
  kv.head_major = head_major;
  if (kv.head_split_changes && head_major) {
    // head-major blocks: a head's tokens are contiguous, so every run of destination heads
    // that sit consecutively on one old rank is one contiguous piece per (layer, K|V, block)
    for (size_t i = 0; i < n_pairs; ++i)
      for (uint32_t rn = 0; rn < kv.d; ++rn) {
        uint32_t hl = 0;
        while (hl < kv.hn) {
          const uint32_t j = rn * kv.hn + hl, ro = kv.src_rank[j], ho = kv.src_head[j];
          uint32_t cnt = 1;
          while (hl + cnt < kv.hn && kv.src_rank[j + cnt] == ro && kv.src_head[j + cnt] == ho + cnt) ++cnt;
          Segment s{};
          s.src_off = pair_old[i] * blk_old + (uint64_t)ho * B * vec;
          s.run_bytes = (uint64_t)cnt * B * vec;
          s.src_pitch = o.kv_num_blocks * blk_old;
          s.n_runs = (uint32_t)(L * 2);
          s.src_rank = ro;
          finish_segment(pp, s, {Dst{pair_new[i] * blk_new + (uint64_t)hl * B * vec,
                                     n.kv_num_blocks * blk_new, rn, 0}});
          hl += cnt;
        }
      }
    pp->bytes_read = per_head * heads_read;  // distinct (old rank, head) slots that are read
    kv.head_split_changes = false;           // the segment kernels do this phase
    return;
  }
  if (kv.head_split_changes) {
    pp->bytes_moved = per_head * kv.d * kv.hn;  // every new rank's heads, replicas included
    pp->bytes_read = per_head * heads_read;     // distinct (old rank, head) slots that are read
    return;
  }
  // head split kept: a block is one contiguous run per (layer, K|V); consecutive
  // pairs that are consecutive in both pools merge into longer runs
  size_t i = 0;
  while (i < n_pairs) {
    size_t j = i + 1;
    while (j < n_pairs && pair_old[j] == pair_old[j - 1] + 1 && pair_new[j] == pair_new[j - 1] + 1)
      ++j;
    for (int t = 0; t < o.tp; ++t) {
      Segment s{};
      s.src_off = pair_old[i] * blk_old;
      s.run_bytes = (uint64_t)(j - i) * blk_old;
      s.src_pitch = o.kv_num_blocks * blk_old;
      s.n_runs = (uint32_t)(L * 2);
      s.src_rank = (uint32_t)t;
      finish_segment(pp, s, {Dst{pair_new[i] * blk_new, n.kv_num_blocks * blk_new, (uint32_t)t, 0}});
    }
    i = j;
  }
}

}  // namespace

uint32_t kv_source_rank(uint32_t hkv, uint32_t c, uint32_t g, uint32_t r_new) {
  const uint32_t h = kv_heads_per_rank(hkv, c);
  auto holds = [&](uint32_t r) {
    const uint32_t f = kv_first_head(hkv, c, r);
    return f <= g && g < f + h;
  };
  if (r_new < c && holds(r_new)) return r_new;  // the same device keeps its copy
  for (uint32_t r = 0; r < c; ++r)
    if (holds(r)) return r;
  return 0;  // not reached for valid degrees
}

// The attention phase again for `replicas` data-parallel copies of the new TP group: every
// segment keeps its source and gets one destination per replica (replica k's rank t is
// new-rank index k * d + t), so a shard is read once however many devices receive it.
void replicate_attn(PhasePlan *pp, int d, uint32_t replicas) {
  if (replicas <= 1) return;
  PhasePlan one = std::move(*pp);
  *pp = PhasePlan();
  pp->arena_old = one.arena_old;
  for (uint32_t k = 0; k < replicas; ++k)
    pp->arena_new.insert(pp->arena_new.end(), one.arena_new.begin(), one.arena_new.end());
  for (const Segment &s0 : one.segs) {
    std::vector<Dst> dsts;
    for (uint32_t k = 0; k < replicas; ++k)
      for (uint32_t j = 0; j < s0.n_dst; ++j) {
        Dst dd = one.dsts[s0.dst_first + j];
        dd.rank += k * (uint32_t)d;
        dsts.push_back(dd);
      }
    Segment s = s0;
    finish_segment(pp, s, dsts);
  }
}

bool phase_is_identity(const PhasePlan &pp) {
  if (pp.arena_old != pp.arena_new) return false;
  for (const Segment &s : pp.segs) {
    if (s.n_dst != 1) return false;
    const Dst &d = pp.dsts[s.dst_first];
    if (d.rank != s.src_rank || d.off != s.src_off || (s.n_runs > 1 && d.pitch != s.src_pitch)) return false;
  }
  return true;
}

emoe_status_t build_host_plan(const emoe_shape_t &sh, const emoe_config_t &o,
                              const emoe_config_t &n, uint32_t flags, uint64_t expert_scale_bytes,
                              uint32_t attn_replicas, HostPlan *hp) {
  if (sh.n_layers <= 0 || sh.n_routed <= 0 || sh.n_shared < 0 || sh.d_model <= 0 ||
      sh.d_ff <= 0 || sh.n_q_heads <= 0 || sh.n_kv_heads <= 0 || sh.head_dim <= 0 ||
      sh.kv_block_tokens <= 0 || sh.elem_bytes <= 0)
    return EMOE_ERR_SHAPE;
  const int n_experts = sh.n_routed + sh.n_shared;
  Placement po, pn;
  emoe_status_t st = read_placement(o, n_experts, &po);
  if (st != EMOE_OK) return st;
  st = read_placement(n, n_experts, &pn);
  if (st != EMOE_OK) return st;
  for (int tp : {o.tp, n.tp}) {
    if (sh.n_q_heads % tp) return EMOE_ERR_SHAPE;
    // more ranks than KV heads: every head is held by tp / Hkv consecutive ranks
    if (tp <= sh.n_kv_heads ? sh.n_kv_heads % tp : tp % sh.n_kv_heads) return EMOE_ERR_SHAPE;
  }
  std::vector<uint32_t> pair_old, pair_new;
  st = read_block_pairs(sh, o, n, &pair_old, &pair_new);
  if (st != EMOE_OK) return st;

  hp->shape = sh;
  hp->ep_old = o.ep; hp->ep_new = n.ep; hp->tp_old = o.tp; hp->tp_new = n.tp;
  plan_experts(sh, po, pn, (uint64_t)sh.d_model * sh.d_ff * sh.elem_bytes, nullptr,
               (flags & EMOE_LAYOUT_FUSED_W13) != 0, expert_scale_bytes, &hp->phase[EMOE_PHASE_EXPERTS]);
  if ((flags & EMOE_LAYOUT_FUSED_QKV) && sh.n_q_heads % sh.n_kv_heads) return EMOE_ERR_SHAPE;
  if (attn_replicas < 1) attn_replicas = 1;
  if ((uint64_t)n.tp * attn_replicas > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  hp->attn_replicas = attn_replicas;
  hp->expert_scale_bytes = expert_scale_bytes;
  plan_attn(sh, o.tp, n.tp, (flags & EMOE_LAYOUT_FUSED_QKV) != 0, &hp->phase[EMOE_PHASE_ATTN]);
  replicate_attn(&hp->phase[EMOE_PHASE_ATTN], n.tp, attn_replicas);
  plan_kv(sh, o, n, std::move(pair_old), std::move(pair_new), (flags & EMOE_LAYOUT_KV_HEAD_MAJOR) != 0, hp);
  for (int ph = 0; ph < 3; ++ph) hp->phase[ph].identity = phase_is_identity(hp->phase[ph]);
  if (hp->kv.head_split_changes) hp->phase[EMOE_PHASE_KV].identity = false;
  return EMOE_OK;
}

emoe_status_t build_paged_expert_plan(const emoe_shape_t &sh, const emoe_config_t &o,
                                      const emoe_config_t &n, uint64_t slab, PhasePlan *pp,
                                      std::vector<Remap> *remaps) {
  if (sh.n_layers <= 0 || sh.n_routed <= 0 || sh.n_shared < 0 || sh.d_model <= 0 || sh.d_ff <= 0 ||
      sh.elem_bytes <= 0)
    return EMOE_ERR_SHAPE;
  if (slab < (uint64_t)sh.d_model * sh.d_ff * sh.elem_bytes) return EMOE_ERR_INVALID_ARG;
  Placement po, pn;
  emoe_status_t st = read_placement(o, sh.n_routed + sh.n_shared, &po);
  if (st != EMOE_OK) return st;
  st = read_placement(n, sh.n_routed + sh.n_shared, &pn);
  if (st != EMOE_OK) return st;
  plan_experts(sh, po, pn, slab, remaps, false, 0, pp);
  return EMOE_OK;
}

emoe_status_t build_inplace_expert_plan(const emoe_shape_t &sh, int ep_old, const int32_t *off_old,
                                        const int32_t *ids_old, int ep_new, const int32_t *cap_new,
                                        const int32_t *want_off, const int32_t *want_ids, uint64_t slab,
                                        PhasePlan *pp, std::vector<std::vector<int32_t>> *slot_new) {
  if (sh.n_layers <= 0 || sh.n_routed <= 0 || sh.n_shared < 0 || sh.d_model <= 0 || sh.d_ff <= 0 ||
      sh.elem_bytes <= 0)
    return EMOE_ERR_SHAPE;
  if (ep_old < 1 || ep_new < 1 || !off_old || !ids_old || !cap_new || !want_off || !want_ids)
    return EMOE_ERR_INVALID_ARG;
  if (ep_old > EMOE_MAX_RANKS || ep_new > EMOE_MAX_RANKS) return EMOE_ERR_UNSUPPORTED;
  const int n_experts = sh.n_routed + sh.n_shared;
  if (off_old[0] != 0 || want_off[0] != 0) return EMOE_ERR_PLACEMENT;
  // old tables: ids in range or -1, an expert at most once per rank
  std::vector<std::pair<int, int>> first_copy(n_experts, {-1, -1});   // smallest (rank, slot)
  for (int r = 0; r < ep_old; ++r) {
    if (off_old[r + 1] < off_old[r]) return EMOE_ERR_PLACEMENT;
    std::vector<char> seen(n_experts, 0);
    for (int i = off_old[r]; i < off_old[r + 1]; ++i) {
      const int32_t e = ids_old[i];
      if (e == -1) continue;
      if (e < 0 || e >= n_experts || seen[e]) return EMOE_ERR_PLACEMENT;
      seen[e] = 1;
      if (first_copy[e].first < 0) first_copy[e] = {r, i - off_old[r]};
    }
  }
  const uint64_t m = (uint64_t)sh.d_model * sh.d_ff * sh.elem_bytes;
  if (slab == 0) slab = m;
  if (slab < m) return EMOE_ERR_INVALID_ARG;
  const uint32_t runs = (uint32_t)sh.n_layers * 3;
  std::vector<uint64_t> slots_old, slots_new;
  for (int r = 0; r < ep_old; ++r) {
    slots_old.push_back((uint64_t)(off_old[r + 1] - off_old[r]));
    pp->arena_old.push_back(runs * slots_old.back() * slab);
  }
  slot_new->assign(ep_new, {});
  std::vector<ExpertMove> moves;
  std::map<std::pair<int, int>, int> fan;
  for (int r = 0; r < ep_new; ++r) {
    if (cap_new[r] < 0 || want_off[r + 1] < want_off[r]) return EMOE_ERR_INVALID_ARG;
    const bool stays = r < ep_old;
    if (stays && (uint64_t)cap_new[r] != slots_old[r]) return EMOE_ERR_INVALID_ARG;  // same arena
    slots_new.push_back((uint64_t)cap_new[r]);
    pp->arena_new.push_back(runs * slots_new.back() * slab);
    std::vector<int32_t> &mine = (*slot_new)[r];
    mine.assign(cap_new[r], -1);
    std::vector<char> free_before(cap_new[r], 1), wanted(n_experts, 0);
    for (int i = want_off[r]; i < want_off[r + 1]; ++i) {
      const int32_t e = want_ids[i];
      if (e < 0 || e >= n_experts || wanted[e]) return EMOE_ERR_PLACEMENT;
      if (first_copy[e].first < 0) return EMOE_ERR_PLACEMENT;   // nobody holds it: it would be lost
      wanted[e] = 1;
    }
    std::vector<char> held(n_experts, 0);
    if (stays)
      for (int s = 0; s < cap_new[r]; ++s) {
        const int32_t e = ids_old[off_old[r] + s];
        if (e < 0) continue;
        free_before[s] = 0;                     // occupied before the step: never overwritten by it
        if (wanted[e]) { mine[s] = e; held[e] = 1; }
      }
    int next_free = 0;
    for (int i = want_off[r]; i < want_off[r + 1]; ++i) {
      const int32_t e = want_ids[i];
      if (held[e]) continue;
      while (next_free < cap_new[r] && !free_before[next_free]) ++next_free;
      if (next_free == cap_new[r]) return EMOE_ERR_TOO_LARGE;
      mine[next_free] = e;
      moves.push_back({first_copy[e].first, first_copy[e].second, r, next_free});
      fan[first_copy[e]]++;
      ++next_free;
    }
  }
  emit_expert_moves(sh, slots_old, slots_new, slab, m, nullptr, nullptr, moves, fan, false, pp);
  return EMOE_OK;
}

void export_segments(const HostPlan &hp, int phase, std::vector<emoe_segment_t> *out) {
  out->clear();
  const PhasePlan &pp = hp.phase[phase];
  uint32_t group = 0;
  for (const Segment &s : pp.segs) {
    for (uint32_t k = 0; k < s.n_dst; ++k) {
      const Dst &d = pp.dsts[s.dst_first + k];
      out->push_back({s.src_off, d.off, s.run_bytes, s.src_pitch, d.pitch, s.n_runs, s.src_rank,
                      d.rank, group});
    }
    ++group;
  }
  if (phase != EMOE_PHASE_KV || !hp.kv.head_split_changes) return;
  const KvPlan &kv = hp.kv;
  const uint64_t hc = kv.hc, hn = kv.hn, B = kv.block_tokens, vec = kv.head_bytes;
  for (size_t i = 0; i < kv.pair_old.size(); ++i)
    for (uint64_t lk = 0; lk < (uint64_t)kv.n_layers * 2; ++lk)
      for (uint32_t rn = 0; rn < kv.d; ++rn) {
        uint32_t hl = 0;
        while (hl < hn) {  // runs of destination heads that are consecutive on one old rank
          const uint32_t j = rn * (uint32_t)hn + hl, ro = kv.src_rank[j], ho = kv.src_head[j];
          uint32_t n = 1;
          while (hl + n < hn && kv.src_rank[j + n] == ro && kv.src_head[j + n] == ho + n) ++n;
          out->push_back({((lk * kv.nb_old + kv.pair_old[i]) * B * hc + ho) * vec,
                          ((lk * kv.nb_new + kv.pair_new[i]) * B * hn + hl) * vec,
                          n * vec, hc * vec, hn * vec, (uint32_t)B, ro, rn, group++});
          hl += n;
        }
      }
}

}  // namespace emoe
