// emoe_oracle.cpp - CPU reference of the scale-step re-layout.
//
// TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's
// CPU-baseline leg may call this file; the product never does.  It shares no
// code, header, table or helper with the CUDA library.
//
// The re-layout reaches a result with a plain definition (a permutation /
// replication of bytes), so this file IS that definition: nested loops over
// logical coordinates in the order the definition states them, one memcpy of
// the innermost contiguous unit, one thread, no segment lists, no coalescing.
//
// Where the definitions come from:
//  * experts: after a scaling step every device holds its experts as one
//    contiguous tensor in slot order (paper Sec. 4.1 "Virtual Expert
//    Management", App. D.5); which experts a device holds is given by the old
//    and new placement (Sec. 5.2 "Expert Weights", App. E for scale-down);
//    uneven and replicated placements are allowed (Sec. 2.1).
//  * attention: TP shards the attention operations (Sec. 2.1); with TP fixed
//    the shards carry over unchanged (Sec. 5.2 "Attention Weights"); changing
//    TP is the paper's future work (App. C "Limitations and Future Work"),
//    read here in the usual way: q/k/v split by head along stored rows, o
//    split by head along stored columns.
//  * KV cache: follows TP (Sec. 4.1, Sec. 5.2 "KV Cache"); "reshaping KV
//    caches" under a TP change (App. C) is read as a contiguous split of the
//    KV heads, block tables translating physical block ids.
//
//  * more TP ranks than KV heads (grouped-query attention; the paper is silent):
//    read in the usual way - with T > Hkv and Hkv | T every KV head is held by
//    T / Hkv consecutive ranks, one head per rank: rank t holds head
//    floor(t * Hkv / T).  Which replica a new rank copies from follows the same
//    rule as for replicated experts: the old rank with the same index if it
//    holds the head, else the smallest old rank that does.
//
//  * layout variants (the paper only says experts are "large contiguous tensors" and
//    KV blocks are paged, Sec. 4.1): fused_w13 stores, per layer, a [n_r][gate|up]
//    tensor followed by a [n_r][down] tensor instead of three [n_r] tensors;
//    head_major stores a KV block as [local head][token][hd] instead of
//    [token][local head][hd].  Both are re-orderings of the same logical data.
//
//  * fused qkv (the paper leaves the attention tensors' form open; serving engines keep
//    one fused projection per rank): the q, k and v rows of a rank form ONE matrix whose
//    rows are grouped by KV head - for every KV head the rank holds, the rows of the
//    query heads of that head's group that the rank holds, then the head's k rows, then
//    its v rows.  With T <= Hkv a rank holds Hkv/T whole groups; with T > Hkv it holds
//    one KV head and Hq/T of its group's query heads.  o is unchanged.
//
//  * quantised experts with block scales (the paper's largest model, Sec. 7.2, ships FP8
//    weights with one scale per 128 x 128 block): every expert matrix has a second, small
//    tensor that must travel with it.  Read here as one arena per rank holding the weight
//    tensor [L][3][n_r][m] and, from the next multiple of 256 bytes on, the scale tensor
//    [L][3][n_r][ms]; both are re-packed by the same placement.
//
//  * in-place expert step (Sec. 4.1 "Virtual Expert Management", Sec. 5.2 "Expert
//    Weights", App. D.5, App. E): a device that stays keeps the experts it already
//    holds where they are and only arrivals are transferred.  Read here for a dense
//    arena with spare capacity, [L][3][cap_r][m] with a slot table (expert id or -1
//    per slot): an expert wanted again keeps its slot; an arrival takes the lowest
//    slot that was FREE BEFORE the step (the old instance keeps serving from the old
//    experts until the switch-over, Sec. 5.2 "Coordinator Performs Instance
//    Switchover", so their bytes are not overwritten); a slot whose expert leaves is
//    marked free for later steps and its bytes stay.
//
// Pins: every function below is pinned by tests that do not use it to make
// their expectation (numpy/torch indexing of logical tensors, hand-written
// fixtures, identities and round trips); none is "parity unpinned".
#include <cstdint>
#include <cstring>

namespace {

struct Csr {
  int n_ranks;
  const int32_t *off;
  const int32_t *ids;
  int count(int r) const { return off[r + 1] - off[r]; }
  int id(int r, int s) const { return ids[off[r] + s]; }
};

// Source replica of expert e for destination rank r_new: the copy held by the
// old rank with the same index if there is one (that device keeps its copy:
// Sec. 5.2 plans a step so that data already in place is reused rather than
// transferred), else the smallest (rank, slot).
bool find_source(const Csr &old_p, int e, int r_new, int *r_out, int *s_out) {
  if (r_new < old_p.n_ranks) {
    for (int s = 0; s < old_p.count(r_new); ++s)
      if (old_p.id(r_new, s) == e) { *r_out = r_new; *s_out = s; return true; }
  }
  for (int r = 0; r < old_p.n_ranks; ++r)
    for (int s = 0; s < old_p.count(r); ++s)
      if (old_p.id(r, s) == e) { *r_out = r; *s_out = s; return true; }
  return false;
}

// KV heads of a TP=T group: heads per rank, first head of rank t, and the old rank
// a new rank takes global head g from (own index first, else the smallest holder).
int64_t kv_heads_per_rank(int64_t hkv, int64_t T) { return hkv >= T ? hkv / T : 1; }
int64_t kv_first_head(int64_t hkv, int64_t T, int64_t t) { return t * hkv / T; }
bool kv_tp_ok(int64_t hkv, int64_t T) { return T >= 1 && (hkv >= T ? hkv % T == 0 : T % hkv == 0); }
int64_t kv_source_rank(int64_t hkv, int64_t c, int64_t g, int64_t r_new) {
  const int64_t h = kv_heads_per_rank(hkv, c);
  if (r_new < c) {
    const int64_t f = kv_first_head(hkv, c, r_new);
    if (f <= g && g < f + h) return r_new;
  }
  for (int64_t r = 0; r < c; ++r) {
    const int64_t f = kv_first_head(hkv, c, r);
    if (f <= g && g < f + h) return r;
  }
  return -1;
}

}  // namespace

extern "C" {

// Bytes of the expert arena of a rank holding n_slots experts: [L][3][n_slots][m].
int64_t emoe_oracle_expert_arena_bytes(int n_layers, int n_slots, int64_t m) {
  return (int64_t)n_layers * 3 * n_slots * m;
}

// Bytes of the attention arena of one TP rank: [L][q_t | k_t | v_t | o_t].
int64_t emoe_oracle_attn_arena_bytes(int n_layers, int d_model, int hq, int hkv, int hd, int b,
                                     int tp) {
  int64_t q = (int64_t)(hq / tp) * hd * d_model * b;
  int64_t kv = kv_heads_per_rank(hkv, tp) * hd * d_model * b;
  return (int64_t)n_layers * (q + 2 * kv + q);
}

// Bytes of the KV arena of one TP rank: [L][2][NB][B][Hkv/T][hd].
int64_t emoe_oracle_kv_arena_bytes(int n_layers, int nb, int block_tokens, int hkv, int hd, int b,
                                   int tp) {
  return (int64_t)n_layers * 2 * nb * block_tokens * kv_heads_per_rank(hkv, tp) * hd * b;
}

// Expert re-pack.  m = bytes of one expert matrix.  Returns 0, or -1 if an
// expert of the new placement has no copy in the old one.
// Offset of matrix (layer l, projection p, slot s) in the arena of a rank with n slots.
// Plain layout: [L][3][n][m].  fused_w13: per layer [n][gate|up] (2m per slot), then [n][down].
int64_t expert_offset(int fused_w13, int64_t l, int p, int64_t n, int64_t s, int64_t m) {
  if (!fused_w13) return ((l * 3 + p) * n + s) * m;
  const int64_t layer = l * 3 * n * m;
  return p < 2 ? layer + s * 2 * m + p * m : layer + n * 2 * m + s * m;
}

int emoe_oracle_reshard_experts(int n_layers, int64_t m, int ep_old, const int32_t *old_off,
                                const int32_t *old_ids, int ep_new, const int32_t *new_off,
                                const int32_t *new_ids, const uint8_t *const *src,
                                uint8_t *const *dst, int fused_w13) {
  Csr po{ep_old, old_off, old_ids}, pn{ep_new, new_off, new_ids};
  for (int rn = 0; rn < ep_new; ++rn) {
    const int64_t n_new = pn.count(rn);
    for (int l = 0; l < n_layers; ++l)
      for (int p = 0; p < 3; ++p)
        for (int sn = 0; sn < n_new; ++sn) {
          int ro, so;
          if (!find_source(po, pn.id(rn, sn), rn, &ro, &so)) return -1;
          const int64_t n_old = po.count(ro);
          const int64_t off_new = expert_offset(fused_w13, l, p, n_new, sn, m);
          const int64_t off_old = expert_offset(fused_w13, l, p, n_old, so, m);
          std::memcpy(dst[rn] + off_new, src[ro] + off_old, (size_t)m);
        }
  }
  return 0;
}

// Attention re-slice TP=c -> TP=d.  b = bytes per element.
int emoe_oracle_reshard_attn(int n_layers, int d_model, int hq, int hkv, int hd, int b, int c,
                             int d, const uint8_t *const *src, uint8_t *const *dst) {
  if (hq % c || hq % d || !kv_tp_ok(hkv, c) || !kv_tp_ok(hkv, d)) return -1;
  const int64_t D = d_model;
  const int64_t row = D * b;  // one stored row of Wq / Wk / Wv
  // sizes of the four pieces of one layer on a rank of a TP=T group
  auto q_bytes = [&](int T) { return (int64_t)(hq / T) * hd * row; };
  auto kv_bytes = [&](int T) { return kv_heads_per_rank(hkv, T) * hd * row; };
  auto layer_bytes = [&](int T) { return 2 * q_bytes(T) + 2 * kv_bytes(T); };

  for (int l = 0; l < n_layers; ++l) {
    // q: global stored row g of the logical matrix
    {
      const int64_t rows = (int64_t)hq * hd;
      const int64_t rows_c = rows / c, rows_d = rows / d;
      for (int64_t g = 0; g < rows; ++g) {
        const int64_t ro = g / rows_c, lo = g % rows_c;
        const int64_t rn = g / rows_d, ln = g % rows_d;
        std::memcpy(dst[rn] + l * layer_bytes(d) + ln * row, src[ro] + l * layer_bytes(c) + lo * row,
                    (size_t)row);
      }
    }
    // k, v: every new rank's local heads, each taken from the old rank chosen for that head
    for (int t = 1; t < 3; ++t) {
      auto piece_off = [&](int T) { return (t == 1) ? q_bytes(T) : q_bytes(T) + kv_bytes(T); };
      for (int rn = 0; rn < d; ++rn)
        for (int64_t hl = 0; hl < kv_heads_per_rank(hkv, d); ++hl) {
          const int64_t g = kv_first_head(hkv, d, rn) + hl;
          const int64_t ro = kv_source_rank(hkv, c, g, rn);
          const int64_t ho = g - kv_first_head(hkv, c, ro);
          for (int64_t r = 0; r < hd; ++r)
            std::memcpy(dst[rn] + l * layer_bytes(d) + piece_off(d) + (hl * hd + r) * row,
                        src[ro] + l * layer_bytes(c) + piece_off(c) + (ho * hd + r) * row, (size_t)row);
        }
    }
    // o: stored row i, head h owns columns [h*hd, (h+1)*hd) of the logical Wo
    const int64_t o_off_c = q_bytes(c) + 2 * kv_bytes(c), o_off_d = q_bytes(d) + 2 * kv_bytes(d);
    const int64_t cols_c = (int64_t)(hq / c) * hd, cols_d = (int64_t)(hq / d) * hd;
    for (int64_t i = 0; i < D; ++i)
      for (int h = 0; h < hq; ++h) {
        const int64_t col = (int64_t)h * hd;
        const int64_t ro = col / cols_c, lo = col % cols_c;
        const int64_t rn = col / cols_d, ln = col % cols_d;
        std::memcpy(dst[rn] + l * layer_bytes(d) + o_off_d + (i * cols_d + ln) * b,
                    src[ro] + l * layer_bytes(c) + o_off_c + (i * cols_c + lo) * b,
                    (size_t)hd * b);
      }
  }
  return 0;
}

// KV head re-split + re-paging.  bt_old / bt_new: [n_seqs][max_blocks].
// Returns 0, or -1 on an unmapped (negative) entry inside a sequence.
int emoe_oracle_reshard_kv(int n_layers, int block_tokens, int hkv, int hd, int b, int c, int d,
                           int nb_old, int nb_new, int n_seqs, int max_blocks,
                           const int32_t *seq_lens, const int32_t *bt_old, const int32_t *bt_new,
                           const uint8_t *const *src, uint8_t *const *dst, int head_major) {
  if (!kv_tp_ok(hkv, c) || !kv_tp_ok(hkv, d)) return -1;
  const int64_t B = block_tokens, hc = kv_heads_per_rank(hkv, c), hdn = kv_heads_per_rank(hkv, d);
  const int64_t vec = (int64_t)hd * b;
  for (int s = 0; s < n_seqs; ++s) {
    const int n_blk = (int)((seq_lens[s] + B - 1) / B);
    for (int j = 0; j < n_blk; ++j) {
      const int64_t po = bt_old[(int64_t)s * max_blocks + j];
      const int64_t pn = bt_new[(int64_t)s * max_blocks + j];
      if (po < 0 || pn < 0 || po >= nb_old || pn >= nb_new) return -1;
      for (int l = 0; l < n_layers; ++l)
        for (int kv = 0; kv < 2; ++kv)
          for (int64_t tok = 0; tok < B; ++tok)
            for (int64_t rn = 0; rn < d; ++rn)
              for (int64_t hn = 0; hn < hdn; ++hn) {
                const int64_t g = kv_first_head(hkv, d, rn) + hn;   // global KV head
                const int64_t ro = kv_source_rank(hkv, c, g, rn);
                const int64_t ho = g - kv_first_head(hkv, c, ro);
                // position of (token, local head) inside a block of H local heads
                auto in_block = [&](int64_t H, int64_t h) { return head_major ? h * B + tok : tok * H + h; };
                const int64_t off_o = ((((int64_t)l * 2 + kv) * nb_old + po) * B * hc + in_block(hc, ho)) * vec;
                const int64_t off_n = ((((int64_t)l * 2 + kv) * nb_new + pn) * B * hdn + in_block(hdn, hn)) * vec;
                std::memcpy(dst[rn] + off_n, src[ro] + off_o, (size_t)vec);
              }
    }
  }
  return 0;
}

// ---- in-place expert step on capacity-strided arenas ---------------------------------
//
// Slot tables are CSR: rank r has slots ids[off[r] .. off[r+1]), each an expert id or -1.
// cap_new[r] is the capacity of new rank r; a rank that exists on both sides keeps its
// arena, so its capacity must not change.  want_off / want_ids: the experts every new rank
// must hold afterwards (order matters only for which free slot an arrival gets).
// Return codes: 0 ok, -1 a wanted expert has no copy in the old tables, -2 a rank has
// fewer free slots than arrivals, -3 a staying rank's capacity differs, -4 a wanted
// expert is listed twice for one rank.

// New slot tables (slot_new: sum(cap_new) entries, rank after rank).
int emoe_oracle_inplace_slots(int ep_old, const int32_t *off_old, const int32_t *ids_old, int ep_new,
                              const int32_t *cap_new, const int32_t *want_off,
                              const int32_t *want_ids, int32_t *slot_new) {
  int64_t base = 0;
  for (int r = 0; r < ep_new; ++r) {
    const int cap = cap_new[r];
    int32_t *mine = slot_new + base;
    base += cap;
    const bool stays = r < ep_old;
    if (stays && off_old[r + 1] - off_old[r] != cap) return -3;
    // 1. start from the old table; remember which slots were free before the step
    for (int s = 0; s < cap; ++s) mine[s] = stays ? ids_old[off_old[r] + s] : -1;
    // 2. experts that are not wanted any more leave (their slot is free from the NEXT step on)
    for (int s = 0; s < cap; ++s) {
      if (mine[s] < 0) continue;
      bool wanted = false;
      for (int i = want_off[r]; i < want_off[r + 1]; ++i) wanted = wanted || want_ids[i] == mine[s];
      if (!wanted) mine[s] = -2;  // leaving: neither an expert nor available to an arrival
    }
    // 3. arrivals, in the order they are listed, take the lowest slot that was free before
    for (int i = want_off[r]; i < want_off[r + 1]; ++i) {
      const int32_t e = want_ids[i];
      for (int k = want_off[r]; k < i; ++k)
        if (want_ids[k] == e) return -4;
      bool held = false;
      for (int s = 0; s < cap; ++s) held = held || mine[s] == e;
      if (held) continue;
      int s = 0;
      while (s < cap && mine[s] != -1) ++s;
      if (s == cap) return -2;
      mine[s] = e;
    }
    for (int s = 0; s < cap; ++s)
      if (mine[s] == -2) mine[s] = -1;
  }
  return 0;
}

// The step itself.  arenas: max(ep_old, ep_new) pointers; arena r is [L][3][cap_r][m] with
// cap_r = old capacity for r < ep_old, cap_new[r] otherwise.  Only arrivals are written.
int emoe_oracle_reshard_experts_inplace(int n_layers, int64_t m, int ep_old, const int32_t *off_old,
                                        const int32_t *ids_old, int ep_new, const int32_t *cap_new,
                                        const int32_t *want_off, const int32_t *want_ids,
                                        const int32_t *slot_new, uint8_t *const *arenas) {
  int64_t base = 0;
  for (int rn = 0; rn < ep_new; ++rn) {
    const int64_t cap = cap_new[rn];
    for (int sn = 0; sn < cap; ++sn) {
      const int32_t e = slot_new[base + sn];
      if (e < 0) continue;
      if (rn < ep_old && ids_old[off_old[rn] + sn] == e) continue;  // kept where it is
      // arrival: smallest (rank, slot) that held e before the step
      int ro = -1, so = -1;
      for (int r = 0; r < ep_old && ro < 0; ++r)
        for (int s = 0; s < off_old[r + 1] - off_old[r]; ++s)
          if (ids_old[off_old[r] + s] == e) { ro = r; so = s; break; }
      if (ro < 0) return -1;
      const int64_t cap_o = off_old[ro + 1] - off_old[ro];
      for (int l = 0; l < n_layers; ++l)
        for (int p = 0; p < 3; ++p)
          std::memcpy(arenas[rn] + (((int64_t)l * 3 + p) * cap + sn) * m,
                      arenas[ro] + (((int64_t)l * 3 + p) * cap_o + so) * m, (size_t)m);
    }
    base += cap;
  }
  (void)want_off; (void)want_ids;
  return 0;
}

// ---- attention with a fused qkv matrix per rank -------------------------------------
//
// Arena of rank t of a TP=T group, per layer: [qkv_t | o_t].  qkv_t has
// (Hq/T + 2 * kvh) * hd rows of D*b bytes, kvh = KV heads per rank, grouped by KV head:
//   group j (KV head kv_first_head(t) + j):  qpg query heads | k head | v head,
//   qpg = (Hq/T) / kvh query heads per group on this rank.
// o_t is stored after it exactly as in the unfused arena.
int emoe_oracle_reshard_attn_fused_qkv(int n_layers, int d_model, int hq, int hkv, int hd, int b, int c,
                                       int d, const uint8_t *const *src, uint8_t *const *dst) {
  if (hq % c || hq % d || hq % hkv || !kv_tp_ok(hkv, c) || !kv_tp_ok(hkv, d)) return -1;
  const int64_t D = d_model, row = D * b, head = (int64_t)hd * row;  // one head's rows, contiguous
  auto kvh = [&](int T) { return kv_heads_per_rank(hkv, T); };
  auto qpg = [&](int T) { return (int64_t)(hq / T) / kvh(T); };
  auto qkv_bytes = [&](int T) { return ((int64_t)(hq / T) + 2 * kvh(T)) * head; };
  auto o_bytes = [&](int T) { return (int64_t)(hq / T) * hd * row; };
  auto layer_bytes = [&](int T) { return qkv_bytes(T) + o_bytes(T); };
  // byte offset, inside a layer of rank (h / (hq/T)), of global query head h
  auto q_off = [&](int T, int64_t h) {
    const int64_t local = h % (hq / T), j = local / qpg(T), i = local % qpg(T);
    return (j * (qpg(T) + 2) + i) * head;
  };
  // ... of the k (which = 0) or v (which = 1) rows of the rank's local KV head j
  auto kv_off = [&](int T, int64_t j, int which) { return (j * (qpg(T) + 2) + qpg(T) + which) * head; };

  for (int l = 0; l < n_layers; ++l) {
    for (int64_t h = 0; h < hq; ++h) {   // query heads: each lives on exactly one rank per side
      const int64_t ro = h / (hq / c), rn = h / (hq / d);
      std::memcpy(dst[rn] + l * layer_bytes(d) + q_off(d, h), src[ro] + l * layer_bytes(c) + q_off(c, h),
                  (size_t)head);
    }
    for (int which = 0; which < 2; ++which)   // k and v heads of every new rank
      for (int rn = 0; rn < d; ++rn)
        for (int64_t jn = 0; jn < kvh(d); ++jn) {
          const int64_t g = kv_first_head(hkv, d, rn) + jn;
          const int64_t ro = kv_source_rank(hkv, c, g, rn);
          const int64_t jo = g - kv_first_head(hkv, c, ro);
          std::memcpy(dst[rn] + l * layer_bytes(d) + kv_off(d, jn, which),
                      src[ro] + l * layer_bytes(c) + kv_off(c, jo, which), (size_t)head);
        }
    // o: exactly as in the unfused arena (stored row i, head h owns columns [h*hd, (h+1)*hd))
    const int64_t cols_c = (int64_t)(hq / c) * hd, cols_d = (int64_t)(hq / d) * hd;
    for (int64_t i = 0; i < D; ++i)
      for (int h = 0; h < hq; ++h) {
        const int64_t col = (int64_t)h * hd;
        const int64_t ro = col / cols_c, lo = col % cols_c;
        const int64_t rn = col / cols_d, ln = col % cols_d;
        std::memcpy(dst[rn] + l * layer_bytes(d) + qkv_bytes(d) + (i * cols_d + ln) * b,
                    src[ro] + l * layer_bytes(c) + qkv_bytes(c) + (i * cols_c + lo) * b, (size_t)hd * b);
      }
  }
  return 0;
}

// ---- experts with a scale tensor per matrix ------------------------------------------
//
// Arena of a rank with n slots: weights [L][3][n][m], then - at the next multiple of 256
// bytes - scales [L][3][n][ms].  Bytes between the two parts belong to nobody.
int64_t emoe_oracle_scaled_expert_scale_base(int n_layers, int n_slots, int64_t m) {
  const int64_t w = (int64_t)n_layers * 3 * n_slots * m;
  return (w + 255) / 256 * 256;
}
int64_t emoe_oracle_scaled_expert_arena_bytes(int n_layers, int n_slots, int64_t m, int64_t ms) {
  return emoe_oracle_scaled_expert_scale_base(n_layers, n_slots, m) + (int64_t)n_layers * 3 * n_slots * ms;
}

int emoe_oracle_reshard_experts_scaled(int n_layers, int64_t m, int64_t ms, int ep_old,
                                       const int32_t *old_off, const int32_t *old_ids, int ep_new,
                                       const int32_t *new_off, const int32_t *new_ids,
                                       const uint8_t *const *src, uint8_t *const *dst) {
  Csr po{ep_old, old_off, old_ids}, pn{ep_new, new_off, new_ids};
  for (int rn = 0; rn < ep_new; ++rn) {
    const int64_t n_new = pn.count(rn);
    const int64_t sb_new = emoe_oracle_scaled_expert_scale_base(n_layers, (int)n_new, m);
    for (int l = 0; l < n_layers; ++l)
      for (int p = 0; p < 3; ++p)
        for (int sn = 0; sn < n_new; ++sn) {
          int ro, so;
          if (!find_source(po, pn.id(rn, sn), rn, &ro, &so)) return -1;
          const int64_t n_old = po.count(ro);
          const int64_t sb_old = emoe_oracle_scaled_expert_scale_base(n_layers, (int)n_old, m);
          const int64_t at_new = ((int64_t)l * 3 + p) * n_new + sn, at_old = ((int64_t)l * 3 + p) * n_old + so;
          std::memcpy(dst[rn] + at_new * m, src[ro] + at_old * m, (size_t)m);                      // the matrix
          std::memcpy(dst[rn] + sb_new + at_new * ms, src[ro] + sb_old + at_old * ms, (size_t)ms);  // its scales
        }
  }
  return 0;
}

}  // extern "C"
