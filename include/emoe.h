/*
 * emoe.h - C ABI of the ElasticMoE scale-step re-layout library (libemoe.so).
 *
 * One scaling step of an elastic MoE serving instance changes the parallel
 * configuration: expert parallelism EP=a -> EP=b and tensor parallelism
 * TP=c -> TP=d.  The paper's HMM derives a redistribution plan from the
 * current and the target configuration (Sec. 5.2 "HMM Reconfigures Memory
 * Layout") and then (i) provisions attention weights, (ii) carries the KV
 * cache over and (iii) migrates experts so that every device again holds
 * its experts as one contiguous tensor (Sec. 4.1 "Virtual Expert
 * Management", App. D.5).  The paper keeps TP fixed and remaps pages instead
 * of copying; it names the copy-based reshaping as the naive alternative
 * (Sec. 4.1) and TP change with KV reshaping as future work (App. C
 * "Limitations and Future Work").  This library implements that copy-based,
 * TP-changing re-layout on ONE GPU, where every "rank" is a distinct region
 * ("arena") of that GPU's memory.
 *
 * All sizes and offsets are in BYTES unless a name says otherwise.  The
 * library never interprets element values; `elem_bytes` only scales sizes.
 *
 * ---------------------------------------------------------------------------
 * Layouts (row-major, densely packed, no padding)
 *
 *   L = n_layers, D = d_model, F = d_ff, b = elem_bytes, hd = head_dim,
 *   Hq = n_q_heads, Hkv = n_kv_heads, B = kv_block_tokens, m = D*F*b.
 *
 *   Experts.  Logical ids 0..n_routed-1 are routed experts, n_routed ..
 *   n_routed+n_shared-1 are shared experts.  The placement of rank r is the
 *   ordered id list P[r] (CSR: place_ids[place_off[r] .. place_off[r+1])),
 *   n_r = |P[r]|.  Expert arena of rank r:
 *        [L][3 (gate, up, down)][n_r][m bytes]
 *   i.e. offset(l, p, s) = ((l*3 + p)*n_r + s) * m.
 *
 *   Attention.  Logical Wq[Hq*hd][D], Wk/Wv[Hkv*hd][D], Wo[D][Hq*hd].
 *   TP=T shard t holds rows [t*Hq*hd/T, (t+1)*Hq*hd/T) of Wq, the same row
 *   slice (over Hkv) of Wk and Wv, and COLUMNS [t*Hq*hd/T, (t+1)*Hq*hd/T) of
 *   Wo.  Attention arena of rank t:  [L][ q_t | k_t | v_t | o_t ], each piece
 *   row-major with its own shard row pitch.
 *
 *   KV cache.  One pool per (layer, K|V) per TP rank, shared block table:
 *        [L][2 (K, V)][kv_num_blocks][B][Hkv/T][hd]
 *   Global KV head g lives on rank g / (Hkv/T) as local head g % (Hkv/T).
 *   With more TP ranks than KV heads (T > Hkv, Hkv | T) every rank holds ONE
 *   head, rank t head floor(t*Hkv/T), so each head is on T/Hkv consecutive
 *   ranks; Wk / Wv rows follow the same rule, Wq / Wo are split T ways.  A new
 *   rank copies a replicated head from the old rank with its own index if that
 *   rank holds the head, else from the smallest old rank that does.
 * ---------------------------------------------------------------------------
 */
#ifndef EMOE_H_
#define EMOE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct emoe_plan emoe_plan_t; /* opaque; owned by the library */

typedef enum {
  EMOE_OK = 0,
  EMOE_ERR_INVALID_ARG = 1,  /* NULL pointer, bad enum value, wrong plan kind         */
  EMOE_ERR_SHAPE = 2,        /* non-positive dimension, TP does not divide the q heads, */
                             /* TP neither divides nor is a multiple of the KV heads    */
  EMOE_ERR_PLACEMENT = 3,    /* id out of range, duplicate inside one rank, expert    */
                             /* missing from the old or from the new placement        */
  EMOE_ERR_BLOCK_TABLE = 4,  /* id out of range, physical block used twice, old/new   */
                             /* sequence sets differ, table shorter than a sequence   */
  EMOE_ERR_ALIGNMENT = 5,    /* an arena base pointer is not 16-byte aligned          */
  EMOE_ERR_OVERLAP = 6,      /* a source arena intersects a destination arena         */
  EMOE_ERR_OOM = 7,          /* host or device allocation for the plan failed         */
  EMOE_ERR_CUDA = 8,         /* a CUDA runtime call failed (no device, bad stream...) */
  EMOE_ERR_UNSUPPORTED = 9,  /* more ranks than EMOE_MAX_RANKS, no virtual memory API   */
  EMOE_ERR_DEVICE_TIMEOUT = 10, /* a bounded device-side wait expired                 */
  EMOE_ERR_TOO_LARGE = 11,   /* the problem exceeds a fixed capacity of the entry point */
  EMOE_ERR_PLAN_CHECK = 12   /* a segment list failed emoe_segments_validate            */
} emoe_status_t;

/* Model shape.  All fields must be > 0 except n_shared (>= 0). */
typedef struct {
  int32_t n_layers;
  int32_t n_routed;        /* routed experts per layer                       */
  int32_t n_shared;        /* shared experts per layer (ids follow routed)   */
  int32_t d_model;
  int32_t d_ff;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;
  int32_t kv_block_tokens; /* tokens per paged-KV block                      */
  int32_t elem_bytes;      /* 2 for bf16                                     */
} emoe_shape_t;

/* One parallel configuration.  Every pointed-to array is caller-owned host
 * memory; emoe_plan_create deep-copies what it needs. */
typedef struct {
  int32_t ep;                 /* expert-parallel ranks (1..EMOE_MAX_RANKS)          */
  int32_t tp;                 /* tensor-parallel ranks (1..EMOE_MAX_RANKS)          */
  const int32_t *place_off;   /* [ep+1] CSR offsets into place_ids                  */
  const int32_t *place_ids;   /* expert ids, rank by rank, in slot order            */
  int32_t kv_num_blocks;      /* physical blocks per (layer, K|V) pool per rank     */
  int32_t n_seqs;             /* sequences in the block table                       */
  int32_t max_blocks;         /* row length of block_table                          */
  const int32_t *seq_lens;    /* [n_seqs] tokens per sequence                       */
  const int32_t *block_table; /* [n_seqs][max_blocks] physical ids, -1 padded       */
} emoe_config_t;

#define EMOE_MAX_RANKS 64

/* emoe_plan_create flags */
#define EMOE_PLAN_HOST_ONLY 1u /* build and validate the plan on the host only: no CUDA */
                               /* call is made, the reshard calls return EMOE_ERR_CUDA  */

#define EMOE_PLAN_HOST_STEP 2u /* also prepare the pipelined form of emoe_reshard_step_host: */
                               /* chunk plans, two copy streams and their events           */

/* Layout variants (the paper fixes neither; Sec. 4.1 only asks for contiguous per-device
 * expert tensors and a paged KV cache).  They apply to BOTH sides of the step. */
#define EMOE_LAYOUT_FUSED_W13 4u     /* expert arena per layer: [n_r][gate|up] (2m per slot),  */
                                     /* then [n_r][down], instead of [3][n_r][m]               */
#define EMOE_LAYOUT_KV_HEAD_MAJOR 8u /* KV block [Hkv/T][B][hd] instead of [B][Hkv/T][hd]     */
#define EMOE_LAYOUT_FUSED_QKV 16u    /* attention arena per layer: [qkv_t | o_t], the rows of  */
                                     /* qkv_t grouped by KV head - for every KV head of the    */
                                     /* rank: the rank's query heads of that head's group,     */
                                     /* then the k head, then the v head (as fused-projection  */
                                     /* checkpoints of grouped-query models store them).       */
                                     /* Needs n_q_heads % n_kv_heads == 0; sizes are unchanged */

/* phase / side selectors of the query helpers */
#define EMOE_PHASE_EXPERTS 0
#define EMOE_PHASE_ATTN 1
#define EMOE_PHASE_KV 2
#define EMOE_PHASE_STEP 3 /* emoe_plan_num_launches only: one emoe_reshard_step call */
#define EMOE_SIDE_OLD 0
#define EMOE_SIDE_NEW 1

/*
 * emoe_plan_create - host planner (Sec. 5.2: the plan is a function of the
 * current and the target configuration only).
 *
 * Validates shape and both configurations, enumerates the logical moves of
 * the three phases, picks the source replica of every destination expert
 * slot (the copy already on the same rank index if there is one, since the
 * paper's plan prefers data that is already on the device to a transfer;
 * otherwise the lexicographically smallest (rank, slot)),
 * coalesces moves into segments, and uploads the descriptor arrays to the
 * current CUDA device (unless EMOE_PLAN_HOST_ONLY).
 *
 * shape, old_cfg, new_cfg: host pointers, read during the call only.
 * n_seqs and seq_lens must agree between old_cfg and new_cfg.
 * out: receives the plan on success, untouched on failure.
 * Errors: any validation failure is reported before any device work.
 */
emoe_status_t emoe_plan_create(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                               const emoe_config_t *new_cfg, uint32_t flags,
                               emoe_plan_t **out);

/*
 * emoe_plan_create_ex - emoe_plan_create with options (NULL options = emoe_plan_create).
 *
 * expert_scale_bytes > 0: every expert matrix travels with a scale tensor of that many
 * bytes - block-quantised weights, as the largest model of the paper's evaluation
 * (Sec. 7.2) ships them: FP8 matrices with one fp32 scale per 128 x 128 block.  The
 * expert arena of a rank with n_r slots is then
 *      weights [L][3][n_r][m]   followed, from the next multiple of 256 bytes on, by
 *      scales  [L][3][n_r][expert_scale_bytes],
 * and ONE plan - one call, one launch set - moves both by the same placement.  Bytes
 * between the two parts are never written.  Not combinable with EMOE_LAYOUT_FUSED_W13
 * (EMOE_ERR_UNSUPPORTED); such a plan's emoe_reshard_step_host runs serially.
 *
 * attn_new_replicas > 1: the new side consists of that many data-parallel replicas of
 * the TP=d group - the paper's attention step (Sec. 5.2 "Attention Weights": devices that
 * are added receive whole copies of the attention tensors from devices that hold them).
 * The attention phase then has tp_new * attn_new_replicas destination arenas, replica
 * after replica (replica k's rank t is index k * tp_new + t), every replica the same
 * re-slice of the old shards; a source run is read ONCE and stored to all replicas.
 * emoe_plan_num_ranks / _arena_bytes report the larger rank count for EMOE_PHASE_ATTN,
 * EMOE_SIDE_NEW, and dst of emoe_reshard_attn / emoe_reshard_step has that many entries.
 * Experts and KV are not affected (a new replica starts with an empty KV cache).
 * tp_new * attn_new_replicas may not exceed EMOE_MAX_RANKS (EMOE_ERR_UNSUPPORTED).
 * 0 and 1 both mean one replica.
 * reserved: must be zero.
 */
typedef struct {
  int64_t expert_scale_bytes;
  int64_t attn_new_replicas;
  int64_t reserved[6];
} emoe_plan_options_t;
emoe_status_t emoe_plan_create_ex(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                                  const emoe_config_t *new_cfg, uint32_t flags,
                                  const emoe_plan_options_t *options, emoe_plan_t **out);

/*
 * emoe_reshard_experts - expert re-pack EP=a -> EP=b (Sec. 4.1 "Virtual
 * Expert Management", Sec. 5.2 "Expert Weights", App. E for b < a).
 *
 * For every new rank r', layer l, projection p and slot s' the matrix of
 * expert P_new[r'][s'] is copied from its source (rank, slot) of the old
 * layout to offset(l, p, s') of the new arena of r'.
 *
 * src: HOST array of ep_old DEVICE pointers (old expert arenas).
 * dst: HOST array of ep_new DEVICE pointers (new expert arenas).
 * cuda_stream: a cudaStream_t (NULL = legacy default stream).
 * Arenas are caller-owned, sized by emoe_plan_arena_bytes, 16-byte aligned,
 * and no source arena may intersect a destination arena (out of place).
 * One exception, the paper's zero-copy case (Sec. 5.2: with TP kept, attention
 * weights and KV cache stay where they are and the new configuration goes on
 * using them): when a phase changes nothing - same rank count, same arena
 * sizes, every byte written comes from the same offset of the same rank index
 * (TP kept and, for the KV cache, block table and pool size kept; for experts,
 * placement kept) - the caller may pass dst[r] == src[r] for EVERY rank (after
 * emoe_plan_set_local_rank: for that rank); the call then returns EMOE_OK and
 * enqueues nothing for that phase.  Any other
 * intersection is still EMOE_ERR_OVERLAP.  emoe_plan_phase_is_identity tells
 * whether a phase qualifies.
 * The call only enqueues work on the stream: it neither synchronises nor
 * allocates.  The pointer arrays are read before the call returns.
 * The device the plan was created on must be the current device of the calling
 * thread (EMOE_ERR_CUDA otherwise, nothing enqueued).
 * Calls may be enqueued on any streams; at most 4 launches of the SAME phase of
 * the SAME plan (a whole-step call counts as a phase of its own) may be
 * enqueued and unfinished at once when they are on different streams (they
 * claim work through per-launch counters of which the plan has 4 per phase,
 * used in turn) - more must be ordered by the caller.  Calls on one stream are always fine.  A call that is
 * being captured into a CUDA graph uses no counter (its CTAs take their work
 * round-robin), so a graph never holds on to one and may be replayed beside
 * live calls.
 */
emoe_status_t emoe_reshard_experts(const emoe_plan_t *plan, const void *const *src,
                                   void *const *dst, void *cuda_stream);

/*
 * emoe_reshard_attn - attention q/k/v/o re-slice TP=c -> TP=d (Sec. 2.1:
 * TP shards the attention operations; Sec. 5.2 "Attention Weights" is the
 * c == d case, a whole-tensor copy onto added devices; App. C names c != d
 * as future work).  q/k/v are split by stored rows (heads), o by stored
 * columns (heads).  src: [tp_old] device pointers, dst: [tp_new]; otherwise
 * as emoe_reshard_experts.
 */
emoe_status_t emoe_reshard_attn(const emoe_plan_t *plan, const void *const *src,
                                void *const *dst, void *cuda_stream);

/*
 * emoe_plan_phase_is_identity - 1 when the phase moves every byte onto its own
 * place (see the zero-copy exception under emoe_reshard_experts; Sec. 5.2),
 * 0 when not, -1 on a bad argument.  Pure host query.
 */
int32_t emoe_plan_phase_is_identity(const emoe_plan_t *plan, int32_t phase);

/*
 * emoe_reshard_kv - paged KV cache head re-split and re-paging (Sec. 5.2
 * "KV Cache" is the c == d, same-table case; App. C "reshaping KV caches").
 *
 * For every sequence s, block index j < ceil(seq_len/B), layer, K|V, token
 * slot and global KV head g, head_dim elements move from old rank
 * g/(Hkv/c), old physical block bt_old[s][j], local head g%(Hkv/c) to new
 * rank g/(Hkv/d), block bt_new[s][j], local head g%(Hkv/d).  Whole blocks
 * move; destination blocks that no sequence maps are not written.
 * src: [tp_old] device pointers, dst: [tp_new]; otherwise as above.
 *
 * Migrating while serving goes on (the paper scales without stopping the old
 * instance, Sec. 4): run the step once for the whole cache, let serving append
 * tokens meanwhile, then run a second, small plan that lists only the blocks
 * written since - each as a "sequence" of one block (seq_len = B, one table
 * entry) - before switching over.  A plan is a pure function of the tables it
 * is given, so any subset of blocks can be re-copied this way.
 */
emoe_status_t emoe_reshard_kv(const emoe_plan_t *plan, const void *const *src,
                              void *const *dst, void *cuda_stream);

/*
 * emoe_reshard_step - the whole scale step (Sec. 5.2: experts, attention
 * weights and KV cache are reconfigured together): the three phases of
 * emoe_reshard_experts / _attn / _kv with the same results, enqueued as at
 * most TWO launches.  The phases touch disjoint arenas, so all their long
 * runs share one launch of the ring kernel (no ramp-up and tail per phase),
 * and what cannot go through the ring - short or strided runs and a KV head
 * re-split - shares one launch of a second kernel.  When both are present the
 * second one is enqueued on a stream that belongs to the plan, forked from
 * cuda_stream and joined back to it with events: it starts after everything
 * cuda_stream held before the call, the two launches run side by side, and
 * cuda_stream continues only after both.  The plan keeps such a stream at
 * the least and at the greatest priority and uses the one nearer to
 * cuda_stream's priority.  The call itself still neither allocates nor
 * synchronises, and it can be captured into a CUDA graph (the plan's stream
 * then belongs to the capture until it ends: make no other whole-step call on
 * that plan meanwhile).  tuning.serial = 1 keeps everything on cuda_stream.
 *
 * src / dst: indexed by EMOE_PHASE_EXPERTS / _ATTN / _KV, each a HOST array of
 * DEVICE pointers as for the per-phase call.  All arguments of all phases are
 * checked before anything is enqueued.  Otherwise as emoe_reshard_experts.
 */
emoe_status_t emoe_reshard_step(const emoe_plan_t *plan, const void *const *const src[3],
                                void *const *const dst[3], void *cuda_stream);

/*
 * emoe_reshard_step_host - one whole scale step on HOST buffers: copies
 * every old arena host->device into caller-provided device staging arenas,
 * runs the three phases, and copies every new arena device->host, all
 * enqueued on cuda_stream (no synchronisation, no allocation).
 *
 * h_src / h_dst: per phase (index EMOE_PHASE_*), HOST arrays of HOST
 * pointers ([ranks of the old side] / [ranks of the new side]); pinned
 * memory is needed for the copies to be asynchronous.
 * d_src / d_dst: per phase, HOST arrays of DEVICE staging pointers with the
 * same rank counts and sizes.  Destination staging arenas are fully
 * overwritten only where the plan writes; bytes the plan does not write are
 * copied back as the staging arena held them.
 *
 * A plan created with EMOE_PLAN_HOST_STEP runs the step as a pipeline over
 * up to 32 chunks of layers (layers are independent in every phase): copy-in of one
 * chunk, the kernels of the previous one and copy-out of the one before
 * overlap on the plan's own two copy streams, so both directions of the host
 * link are busy at once.  Work still starts after what cuda_stream held before
 * the call and cuda_stream ends after the last copy-out.  Calls of this form on
 * ONE plan must not overlap each other (they share the plan's events).  Without
 * the flag, or when a layer slice of an arena is not 16-byte aligned, the step
 * runs serially on cuda_stream alone.
 */
emoe_status_t emoe_reshard_step_host(const emoe_plan_t *plan, const void *const *const h_src[3],
                                     void *const *const h_dst[3],
                                     void *const *const d_src[3], void *const *const d_dst[3],
                                     void *cuda_stream);

/*
 * emoe_reshard_kv_static - the KV head re-split and re-paging of
 * emoe_reshard_kv for callers that must not allocate device memory.  (The
 * paper has no counterpart: this entry point exists for integration only.)
 *
 * Who needs it: a serving process whose memory daemon has already claimed
 * all of HBM for weights and KV pools, so that a cudaMalloc at scaling time
 * would fail or evict something; a caller inside a latency-critical section
 * where the implicit device synchronisation of cudaMalloc / cudaFree is not
 * acceptable; code running under an allocator hook that forbids raw CUDA
 * allocations.  Such a caller creates its plan with EMOE_PLAN_HOST_ONLY
 * (which makes no CUDA call at all) and uses this entry point, which calls
 * no cudaMalloc, no cudaFree and no allocating library routine.
 *
 * The block-pair list the kernel reads (8 bytes per mapped block) is kept in
 * a fixed array inside the library image instead: EMOE_STATIC_KV_MAX_PAIRS
 * pairs = 512 KiB, resident on every GPU that loads libemoe.so until the
 * process exits.  A plan with more mapped blocks is rejected with
 * EMOE_ERR_TOO_LARGE before anything is enqueued.
 *
 * plan: any plan, host-only or not.  src / dst / cuda_stream: exactly as for
 * emoe_reshard_kv (HOST arrays of tp_old / tp_new DEVICE pointers), with the
 * same alignment and no-overlap rules; the result is byte-identical to
 * emoe_reshard_kv, whether or not the TP degree changes.
 *
 * Each call first copies the plan's pair list into the fixed array on
 * cuda_stream, then launches the kernel on the same stream.  The list lives
 * in ordinary (pageable) host memory of the plan, so the driver stages that
 * copy and the CALL may wait until cuda_stream has reached it - up to two
 * copies of 256 KiB; the plan must stay alive until the stream has passed the
 * call.  With emoe_plan_set_local_rank in force only that rank's blocks are
 * written, as for emoe_reshard_kv (other dst[] entries may then be NULL).  All calls on a
 * device share that one array, and it keeps the previous call's list: two
 * calls whose GPU work can overlap (different streams without an ordering
 * between them) race on it and must be serialised by the caller.  Nothing in
 * the array has to start at zero; each call overwrites the prefix it reads.
 *
 * Plans made with EMOE_LAYOUT_KV_HEAD_MAJOR are accepted while the TP degree
 * is kept (whole blocks move); with a changed TP degree they are rejected
 * with EMOE_ERR_UNSUPPORTED, since this entry point has only the token-major
 * re-split kernel.
 *
 * The first call on each device looks up the array's device address
 * (one-time set-up, with that device current).  Make that first call outside
 * any stream capture.
 */
#define EMOE_STATIC_KV_MAX_PAIRS 65536
emoe_status_t emoe_reshard_kv_static(const emoe_plan_t *plan, const void *const *src,
                                     void *const *dst, void *cuda_stream);

/* ---- in-place expert step: only arrivals move -------------------------------
 *
 * The paper's expert step leaves what a device already holds where it is and
 * transfers only the experts that arrive (Sec. 4.1 "Virtual Expert
 * Management", Sec. 5.2 "Expert Weights", App. D.5; App. E for scale-down).
 * This is that step for DENSE arenas with spare capacity - no page re-mapping:
 *
 *   arena of device r:  [L][3 (gate, up, down)][cap_r][m bytes],
 *   slot table of device r: cap_r entries, an expert id or -1 (free).
 *
 * An expert that device r holds and still wants keeps its slot and is not
 * touched.  An arrival is copied from the smallest (device, slot) that held it
 * before the step into the lowest slot of r that was FREE BEFORE the step,
 * arrivals being served in the order want_ids lists them.  A slot whose expert
 * is no longer wanted becomes free in the new table, but its bytes stay: the
 * old instance keeps serving from them until the switch-over (Sec. 5.2), and
 * only a later step may reuse the slot.  So no byte that anything still reads
 * is ever overwritten, and source and destination may be the same arena.
 *
 * emoe_plan_create_inplace
 *   slot_off_old [ep_old+1], slot_ids_old: CSR slot tables before the step
 *     (capacity of device r = slot_off_old[r+1] - slot_off_old[r]).
 *   cap_new [ep_new]: capacities after the step; for r < ep_old it must equal the
 *     old capacity (the device keeps its arena), for an added device it is free.
 *   want_off [ep_new+1], want_ids: the experts every device must hold afterwards.
 *   flags: 0 or EMOE_PLAN_HOST_ONLY.
 *   Errors: EMOE_ERR_PLACEMENT (id out of range, an expert twice in one table or
 *   one want list, a wanted expert nobody holds), EMOE_ERR_TOO_LARGE (a device
 *   has fewer slots free before the step than arrivals), EMOE_ERR_INVALID_ARG
 *   (a staying device's capacity differs), EMOE_ERR_UNSUPPORTED (too many ranks).
 *   The plan answers emoe_plan_stats / _arena_bytes / _num_launches / _segments for
 *   EMOE_PHASE_EXPERTS (bytes_moved = arrivals only; arena sizes by capacity) and
 *   takes emoe_plan_set_tuning / _set_local_rank; it has no attention or KV phase
 *   and the out-of-place reshard calls reject it with EMOE_ERR_INVALID_ARG.
 *
 * emoe_plan_slot_table: the slot table of `rank` after the step (up to `cap`
 *   entries into `out`, the table's length into *n_slots).
 *
 * emoe_reshard_experts_inplace: arenas = HOST array of max(ep_old, ep_new)
 *   DEVICE pointers, arena r serving as source (r < ep_old) and as destination
 *   (r < ep_new).  16-byte aligned; arenas of different devices must not
 *   intersect.  Enqueues on cuda_stream only, like emoe_reshard_experts.
 */
emoe_status_t emoe_plan_create_inplace(const emoe_shape_t *shape, int32_t ep_old,
                                       const int32_t *slot_off_old, const int32_t *slot_ids_old,
                                       int32_t ep_new, const int32_t *cap_new,
                                       const int32_t *want_off, const int32_t *want_ids,
                                       uint32_t flags, emoe_plan_t **out);
emoe_status_t emoe_plan_slot_table(const emoe_plan_t *plan, int32_t rank, int32_t *out, int32_t cap,
                                   int32_t *n_slots);
emoe_status_t emoe_reshard_experts_inplace(const emoe_plan_t *plan, void *const *arenas,
                                           void *cuda_stream);

/* ---- paged expert store: re-layout by re-mapping pages ---------------------
 *
 * The paper's own expert mechanism (Sec. 4.1 "Virtual Expert Management",
 * App. D.5): every expert matrix lives in physical pages of its own, which
 * are mapped into one contiguous virtual range per device; changing the
 * expert-parallel degree re-maps the pages a device keeps and transfers only
 * the experts that arrive.  Here on the CUDA virtual memory API, all ranks
 * being ranges of ONE GPU.
 *
 * Layout of the range of rank r: [L][3 (gate, up, down)][n_r][slab], where
 * slab = one matrix (m bytes) rounded up to the device's allocation
 * granularity (2 MiB on B200); the first m bytes of a slab hold the matrix,
 * the rest is padding.  Apart from the padding this is the dense expert arena.
 */
typedef struct emoe_vmm_pool emoe_vmm_pool_t; /* opaque; owns ranges and pages */

typedef struct {
  uint64_t slabs_remapped; /* (layer, projection, slot) slabs kept by re-mapping        */
  uint64_t slabs_copied;   /* slabs newly allocated and filled by the copy kernels      */
  uint64_t bytes_copied;   /* bytes written by the copy kernels (arrivals only)         */
  uint64_t bytes_read;     /* bytes they read (a source with several arrivals: once)    */
  uint64_t slab_bytes, matrix_bytes;
  uint64_t physical_bytes; /* device memory the pool holds after the step               */
  double map_ms;           /* host time: reserve ranges, allocate and map slabs, enable */
                           /* access; alloc_ms and access_ms are parts of it            */
  double alloc_ms;         /* ... of which allocating the arrivals' physical pages      */
  double access_ms;        /* ... of which enabling access to the new ranges            */
  double copy_ms;          /* host time: plan upload, copy kernels, stream synchronise  */
  double unmap_ms;         /* host time: unmap and free the old ranges, release pages   */
  double total_ms;
} emoe_vmm_stats_t;

/* Allocates the store for the placement of `cfg` (ep, place_off, place_ids;
 * the other fields are ignored) on the current device.  Contents are
 * undefined until written.  EMOE_ERR_UNSUPPORTED if the driver's virtual
 * memory API is not available; EMOE_ERR_OOM if pages or address space run out. */
emoe_status_t emoe_vmm_create(const emoe_shape_t *shape, const emoe_config_t *cfg,
                              emoe_vmm_pool_t **out);

/* Scale step EP=a -> EP=b in place of emoe_reshard_experts: afterwards the
 * pool holds the placement of new_cfg.  A destination slot whose expert the
 * same rank index already holds is re-mapped (no bytes move); every other
 * slot gets fresh pages filled from its source replica (same source rule as
 * emoe_plan_create) by the copy kernels on cuda_stream.  The call is
 * SYNCHRONOUS: it returns after the copies have finished and the old ranges
 * have been unmapped, so every pointer obtained from emoe_vmm_arena before
 * the call is invalid after it.  On failure the pool is unchanged.
 * stats: optional, filled on success. */
emoe_status_t emoe_vmm_reshard(emoe_vmm_pool_t *pool, const emoe_config_t *new_cfg,
                               void *cuda_stream, emoe_vmm_stats_t *stats);

/* What emoe_vmm_reshard would do for old_cfg -> new_cfg with slabs of
 * slab_bytes (>= one matrix), computed on the host without any CUDA call:
 * fills slabs_remapped, slabs_copied, bytes_copied, bytes_read, slab_bytes,
 * matrix_bytes and physical_bytes (of the new placement); times stay 0. */
emoe_status_t emoe_vmm_dry_run(const emoe_shape_t *shape, const emoe_config_t *old_cfg,
                               const emoe_config_t *new_cfg, uint64_t slab_bytes,
                               emoe_vmm_stats_t *stats);

/* Number of ranks / the range of one rank: DEVICE base pointer, its size,
 * the slab stride, the matrix size and the slot count.  NULL outputs are skipped. */
emoe_status_t emoe_vmm_num_ranks(const emoe_vmm_pool_t *pool, int32_t *n);
emoe_status_t emoe_vmm_arena(const emoe_vmm_pool_t *pool, int rank, void **base, uint64_t *bytes,
                             uint64_t *slab_bytes, uint64_t *matrix_bytes, int32_t *n_slots);

/* Copies a DENSE host image [L][3][n_r][m] of rank `rank` into / out of its
 * paged range (asynchronous on cuda_stream; pinned memory to overlap). */
emoe_status_t emoe_vmm_write(emoe_vmm_pool_t *pool, int rank, const void *host_dense,
                             void *cuda_stream);
emoe_status_t emoe_vmm_read(const emoe_vmm_pool_t *pool, int rank, void *host_dense,
                            void *cuda_stream);

/* Unmaps and frees everything (synchronises the device first).  NULL-safe. */
void emoe_vmm_destroy(emoe_vmm_pool_t *pool);

/* ---- paged expert store with slot tables: a step touches only what changes ---
 *
 * The store above builds every range anew at every step.  This variant keeps a device's
 * range for as long as the device exists and follows the in-place expert step
 * (emoe_plan_create_inplace: same slot tables, same rules): the range of device r is
 * RESERVED for cap_r slots, [L][3][cap_r][slab], and only occupied slots have pages.  A
 * step leaves kept experts alone (no driver call, no copy), maps pages into the slots of
 * arrivals - taken from a list of spare pages, so that no physical memory is created
 * inside a step as long as the list lasts - fills them with the copy kernels, and after
 * the copies unmaps the slots of experts that left, whose pages go back to the spare
 * list.  Driver work and bytes copied are proportional to the slots that change.
 *
 * emoe_vmm_slots_create: slot_off [ep+1] / slot_ids: CSR slot tables (-1 = free; capacity
 *   of device r = slot_off[r+1] - slot_off[r]); spare_slots: slots' worth of physical pages
 *   (3 * n_layers slabs each) created up front for the arrivals of later steps.
 * emoe_vmm_slots_reshard: cap_new / want_off / want_ids as for emoe_plan_create_inplace
 *   (same errors, reported before anything is touched).  SYNCHRONOUS: returns after the
 *   copies and the unmapping.  On failure the store is unchanged.  stats (optional):
 *   slabs_remapped counts slabs kept in place, slabs_copied those of arrivals.
 * emoe_vmm_slots_info: base address, capacity and slot table of `rank` (rank < 0: only the
 *   pool-wide outputs: slab size, device count, spare slabs).  NULL outputs are skipped.
 *   A free slot has NO memory behind it: only occupied slots may be read or written.
 * emoe_vmm_slots_write / _read: one occupied slot as a dense host image [L][3][m].
 * emoe_vmm_slots_destroy: synchronises the device, unmaps and frees everything. */
typedef struct emoe_vmm_slots emoe_vmm_slots_t;
emoe_status_t emoe_vmm_slots_create(const emoe_shape_t *shape, int32_t ep, const int32_t *slot_off,
                                    const int32_t *slot_ids, int32_t spare_slots,
                                    emoe_vmm_slots_t **out);
emoe_status_t emoe_vmm_slots_reshard(emoe_vmm_slots_t *pool, int32_t ep_new, const int32_t *cap_new,
                                     const int32_t *want_off, const int32_t *want_ids,
                                     void *cuda_stream, emoe_vmm_stats_t *stats);
emoe_status_t emoe_vmm_slots_info(const emoe_vmm_slots_t *pool, int32_t rank, void **base,
                                  uint64_t *slab_bytes, int32_t *cap, int32_t *ids_out,
                                  int32_t ids_cap, int32_t *n_ranks, int64_t *spare_slabs);
emoe_status_t emoe_vmm_slots_write(emoe_vmm_slots_t *pool, int32_t rank, int32_t slot,
                                   const void *host, void *cuda_stream);
emoe_status_t emoe_vmm_slots_read(const emoe_vmm_slots_t *pool, int32_t rank, int32_t slot,
                                  void *host, void *cuda_stream);
void emoe_vmm_slots_destroy(emoe_vmm_slots_t *pool);

/* emoe_plan_destroy - frees host state and device descriptor buffers.
 * NULL-safe.  No kernel using the plan may still be in flight. */
void emoe_plan_destroy(emoe_plan_t *plan);

/* ---- query helpers ------------------------------------------------------ */

/* Number of ranks on one side of a phase (EP for experts, TP otherwise). */
emoe_status_t emoe_plan_num_ranks(const emoe_plan_t *plan, int phase, int side, int32_t *n);

/* Arena size in bytes of `rank` for (phase, side). */
emoe_status_t emoe_plan_arena_bytes(const emoe_plan_t *plan, int phase, int side, int rank,
                                    uint64_t *bytes);

/* bytes_moved: bytes the phase writes to the new layout.  bytes_read: bytes
 * it reads from the old layout (smaller when one source run feeds several
 * destinations).  n_segments: descriptors after coalescing. */
emoe_status_t emoe_plan_stats(const emoe_plan_t *plan, int phase, uint64_t *bytes_moved,
                              uint64_t *bytes_read, uint64_t *n_segments);

/* Kernel launches one reshard call of this phase enqueues with the current tuning. */
emoe_status_t emoe_plan_num_launches(const emoe_plan_t *plan, int phase, int32_t *n);

/* Work items one reshard call of this phase (or EMOE_PHASE_STEP: one emoe_reshard_step
 * call) hands to each kind of kernel with the current tuning: units of the ring kernel
 * (cp.async.bulk through shared memory), units of the vector kernel, tiles of the KV head
 * re-split (0 when the head split is kept: whole blocks then move as ring or vector units).
 * NULL outputs are skipped.  For reports: which kernels a launch set consists of. */
emoe_status_t emoe_plan_launch_work(const emoe_plan_t *plan, int phase, uint64_t *ring_units,
                                    uint64_t *vector_units, uint64_t *kv_tiles);

/* One coalesced copy descriptor, as exported for inspection and host-side
 * replay: n_runs runs of run_bytes each; run i reads
 * src[src_rank] + src_off + i*src_pitch and writes
 * dst[dst_rank] + dst_off + i*dst_pitch.  A source run that feeds several
 * destinations appears once per destination with the same `group` value. */
typedef struct {
  uint64_t src_off, dst_off, run_bytes, src_pitch, dst_pitch;
  uint32_t n_runs, src_rank, dst_rank, group;
} emoe_segment_t;

/* Copies up to `cap` segments of the phase into `out` (host memory) and
 * stores the total count in *n.  For a KV phase that changes the head split
 * the block-pair list is expanded into one segment per (pair, layer, K|V,
 * old rank, new rank) overlap, its runs being the block's token rows. */
emoe_status_t emoe_plan_segments(const emoe_plan_t *plan, int phase, emoe_segment_t *out,
                                 uint64_t cap, uint64_t *n);

/* emoe_segments_validate / emoe_plan_validate - the host-side bounds and race check.
 * Copy kernels can only fault by leaving an arena and only race by writing one byte twice;
 * both are properties of the segment list.  Checks, for segments as emoe_plan_segments
 * exports them and arena sizes in bytes: every source run and every destination run lies
 * inside its arena (ranks in range, no arithmetic overflow), a segment's own runs do not
 * overlap, destination runs of one arena are pairwise disjoint, and - with must_tile - they
 * cover the arena exactly (weights: every byte of a new arena is written once).
 * Returns EMOE_OK or EMOE_ERR_PLAN_CHECK with the index of an offending segment in
 * *bad_segment (optional; n_segs if an arena's tail is not covered).  Host only.
 * emoe_plan_validate runs it on a plan's own three phases (experts and attention must tile;
 * the KV phase need not: unmapped blocks are not written; an in-place plan must not tile
 * either: kept slots are not written) and stores the failing phase in *bad_phase.  A plan made
 * by this library passes; the call exists for callers that want the guarantee re-checked
 * (after an upgrade, under test) and costs time proportional to the number of runs. */
emoe_status_t emoe_segments_validate(const emoe_segment_t *segs, uint64_t n_segs,
                                     const uint64_t *arena_old, int32_t n_old,
                                     const uint64_t *arena_new, int32_t n_new, int32_t must_tile,
                                     uint64_t *bad_segment);
emoe_status_t emoe_plan_validate(const emoe_plan_t *plan, int32_t *bad_phase, uint64_t *bad_segment);

/* Reads the plan's device status word (EMOE_OK or EMOE_ERR_DEVICE_TIMEOUT).
 * Synchronises the device copy on the legacy default stream; call it after
 * the caller has synchronised the stream(s) the plan ran on. */
emoe_status_t emoe_plan_device_status(const emoe_plan_t *plan, int32_t *status);

/* Clears the status word after an EMOE_ERR_DEVICE_TIMEOUT has been read; the plan is
 * usable again (the launch that timed out has left its destination undefined).  Call it
 * with none of the plan's launches in flight. */
emoe_status_t emoe_plan_clear_device_status(emoe_plan_t *plan);

/* Launch tuning.  Fields set to 0 keep the library default. */
typedef struct {
  int32_t max_ctas;        /* upper bound on CTAs per launch (SM budget when the    */
                           /* reshard shares the GPU with a live kernel).  The ring */
                           /* kernel keeps one CTA per SM for the whole launch and  */
                           /* a live kernel loses those SMs: 16 keeps a concurrent  */
                           /* GEMM within 1.5x on B200; more than the default (74)  */
                           /* and fewer than all SMs only hurts both sides.  (path  */
                           /* = 3 takes no SM at all, at the copy engines' rate.)   */
  int32_t bulk_tile_bytes; /* bytes per shared-memory stage of the bulk kernel      */
  int32_t bulk_stages;     /* stages of the bulk kernel's ring                      */
  int32_t path;            /* 0 default routing, 1 force the vector kernel for all  */
                           /* segments, 2 force the bulk kernel where aligned, 3    */
                           /* one driver copy (cudaMemcpy2DAsync, copy engines) per */
                           /* segment and destination instead of the kernels - no   */
                           /* SM is taken from a kernel that runs beside it; a KV   */
                           /* head re-split still uses its kernel                   */
  int32_t kv_mode;         /* 0 default, 1 direct, 2 staged through shared memory,  */
                           /* 3 tiled TMA loads and stores, 4 direct without the    */
                           /* row-mapped fast path                                  */
  int32_t bulk_hints;      /* 0 default, 1 none, 2 loads evict-first in L2, 3 stores */
                           /* evict-first, 4 both                                   */
  int32_t kv_order;        /* order in which mapped KV blocks are visited: 0 default    */
                           /* (= 2), 1 block-table order, 2 by old physical id (reads   */
                           /* walk the old pool in address order), 3 by new id          */
  int32_t unit_order;      /* bulk work order: 0 default (run-major: one layer slab or  */
                           /* KV pool at a time), 1 segment-major; +2: CTAs take units  */
                           /* round-robin instead of claiming them from a counter       */
  int32_t wait_limit_us;   /* bound of every device-side wait in microseconds (default  */
                           /* 4 s).  -1: a wait that is not already satisfied when it   */
                           /* is first polled expires at once - for exercising the      */
                           /* time-out path; such a launch returns normally, sets the   */
                           /* status word and leaves its destination undefined          */
  int32_t bw_limit_gbs;    /* bandwidth limit of the ring kernel in GB/s of bytes read  */
                           /* plus bytes written (its CTAs space their loads so that    */
                           /* the launch as a whole stays near it); 0 = none.  For a    */
                           /* reshard that shares HBM with a live kernel                */
  int32_t bulk_min_run;    /* 16-byte-aligned runs of at least this many bytes go to    */
                           /* the ring kernel (default 16384; a multiple of 16)         */
  int32_t serial;          /* emoe_reshard_step: 1 = its launch sets run one after the  */
                           /* other on the caller's stream; 2 = also keep the vector    */
                           /* work and the KV head re-split in separate kernels         */
} emoe_tuning_t;

/* Replaces the plan's launch tuning.  Not thread-safe against reshard calls
 * running concurrently on other host threads. */
emoe_status_t emoe_plan_set_tuning(emoe_plan_t *plan, const emoe_tuning_t *tuning);

/* emoe_place_min_transfer - a placement for EP=ep_new that keeps as many experts
 * where they are as balance allows (Sec. 5.2 "Expert Weights": the new placement
 * balances the experts while moving as little as possible; the paper gives no
 * algorithm).  Every expert 0..n_experts-1 is placed exactly once, rank sizes
 * differ by at most one, slots within a rank are in id order, and the number of
 * experts placed on a rank index that already holds a copy in old_cfg (ep,
 * place_off, place_ids; other fields ignored) is the maximum any such placement
 * reaches.  Experts that have to move fill the free slots in id order.
 * new_off: [ep_new + 1], new_ids: [n_experts], caller-owned host arrays;
 * n_kept (optional): the number of experts that stay.  Host only, no CUDA call. */
emoe_status_t emoe_place_min_transfer(int32_t n_experts, const emoe_config_t *old_cfg,
                                      int32_t ep_new, int32_t *new_off, int32_t *new_ids,
                                      int32_t *n_kept);

/* ---- plans for scaling sequences ------------------------------------------
 *
 * A serving system that scales up and down in steps (the paper's step patterns add or
 * remove devices a few at a time, Sec. 7.4; scale-down mirrors scale-up, App. E) meets
 * the same (old, new) pairs again.  A plan is a pure function of its inputs, so a cache
 * can hand out the plan made earlier: emoe_plan_cache_get returns the cached plan when
 * shape, flags, options and everything emoe_plan_create reads from the two configurations
 * (placements, TP/EP degrees, pool sizes, sequence lengths, the mapped block-table
 * entries) are byte-for-byte the same, and otherwise creates one (on the current CUDA
 * device unless EMOE_PLAN_HOST_ONLY; the device is part of the key) and keeps it.
 * *hit (optional): 1 / 0.
 * The cache OWNS its plans: never pass them to emoe_plan_destroy.  It keeps at most
 * `capacity` plans; inserting one more destroys the least recently used one, so a plan
 * obtained earlier may die in a later emoe_plan_cache_get - do not hold more plans than
 * the capacity across calls, and have no launch of an evicted plan in flight.
 * Invalid inputs return the planner's error and are not stored.  Thread-safe.
 * Weights and KV can be cached separately: a plan whose configurations list no sequences
 * (n_seqs = 0) covers experts and attention and does not depend on block tables. */
typedef struct emoe_plan_cache emoe_plan_cache_t;
emoe_status_t emoe_plan_cache_create(int32_t capacity, emoe_plan_cache_t **out);
emoe_status_t emoe_plan_cache_get(emoe_plan_cache_t *cache, const emoe_shape_t *shape,
                                  const emoe_config_t *old_cfg, const emoe_config_t *new_cfg,
                                  uint32_t flags, const emoe_plan_options_t *options,
                                  emoe_plan_t **plan, int32_t *hit);
emoe_status_t emoe_plan_cache_stats(emoe_plan_cache_t *cache, uint64_t *hits, uint64_t *misses,
                                    uint64_t *evictions, int32_t *size);
void emoe_plan_cache_destroy(emoe_plan_cache_t *cache);

/* emoe_kv_compact_table - a destination block table that COMPACTS the cache while it
 * moves: the mapped blocks of the sequences, in table order (sequence by sequence, block
 * by block), get the lowest-numbered blocks of the destination pool that are free.  The
 * paper leaves block allocation across the two instances open (App. C names coordinating
 * it as future work); this is the allocation a scale-down wants, where the surviving pool
 * should end up dense.
 * in_use [n_in_use]: blocks of the destination pool (size nb_new) that are already taken -
 * e.g. by sequences the new instance serves already - and must not be handed out; NULL /
 * 0 for a fresh pool, which yields the identity order 0, 1, 2, ...
 * old_table (optional, [n_seqs][max_blocks]): the table the blocks are read through.  If
 * given, the blocks are served in the order of their OLD physical id instead of table order:
 * the free ids are the same, but old and new addresses then rise together, and a migration
 * - which visits the blocks in old-pool order - reads AND writes in address order (measured
 * on B200: the KV phase 0.8 to 1.3 % faster than with the ids handed out in table order).
 * table_out: [n_seqs][max_blocks], -1 padded; *n_mapped (optional): blocks assigned.
 * Errors: EMOE_ERR_BLOCK_TABLE (an in_use id out of range or listed twice, a sequence
 * longer than max_blocks blocks, an unmapped old entry), EMOE_ERR_TOO_LARGE (not enough free
 * blocks).  Host only.  Use the result as new_cfg->block_table of emoe_plan_create. */
emoe_status_t emoe_kv_compact_table(int32_t block_tokens, int32_t n_seqs, int32_t max_blocks,
                                    const int32_t *seq_lens, int32_t nb_new, const int32_t *in_use,
                                    int32_t n_in_use, const int32_t *old_table, int32_t *table_out,
                                    int32_t *n_mapped);

/* ---- one rank per GPU: pull-based exchange --------------------------------
 *
 * With rank = GPU, every destination arena is written by the GPU that owns it
 * and every segment has one source rank, so a scale step is ONE exchange: each
 * GPU pulls what it needs from its peers' old arenas (the counterpart of the
 * paper's P2P transfers, Sec. 4 and App. D) and copies the rest locally.  The
 * kernels are the same; a remote source is simply a peer-mapped pointer.
 *
 * emoe_plan_set_local_rank: from now on the reshard calls of this plan write
 * ONLY the destination arenas of new-rank index `rank` (-1: all, the
 * default).  dst[] entries of other ranks and src[] entries of old ranks that
 * this rank reads nothing from may then be NULL.  Every process builds the
 * same plan from the same configurations and sets its own rank; the union of
 * what the ranks write is the whole step.  Not for plans created with
 * EMOE_PLAN_HOST_STEP.  Synchronises the device (descriptor tables are
 * rebuilt). */
emoe_status_t emoe_plan_set_local_rank(emoe_plan_t *plan, int32_t rank);

/* Sharing an arena with the other processes of the node (CUDA IPC).
 * emoe_ipc_export: handle_out receives EMOE_IPC_HANDLE_BYTES bytes naming the
 * ALLOCATION that contains device_ptr, offset_out the pointer's offset in it.
 * emoe_ipc_open (in another process, with its device current): maps that
 * allocation and returns its base; the arena is at base + offset.
 * emoe_ipc_close: unmaps it.  A process uses its own arenas directly. */
#define EMOE_IPC_HANDLE_BYTES 64
emoe_status_t emoe_ipc_export(const void *device_ptr, void *handle_out, uint64_t *offset_out);
emoe_status_t emoe_ipc_open(const void *handle, void **base_out);
emoe_status_t emoe_ipc_close(void *base);

/* Static string for a status code. */
const char *emoe_strerror(emoe_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* EMOE_H_ */
