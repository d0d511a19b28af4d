/*
 * omnitide.h -- C ABI of the B200 (sm_100a) per-chunk hot path of the OmniTide streaming loop.
 *
 * One pass per incoming chunk and per layer:
 *     score units -> select units -> compact KV (OmniPage) -> append chunk -> chunk-prefill attention
 *
 * Conventions (all entry points)
 *   - C99 ABI, no exceptions.  Every call returns an omni_status.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue device work on it and return; none
 *     of them synchronises the host.  Errors the host can see (null / misaligned pointers, unsupported
 *     geometry, capacity) are returned at once; errors found on the device (a bounded wait that ran
 *     out, a malformed unit table) are OR-ed into a status word read with omnitide_poll_status().
 *   - Pointers marked [dev] are device pointers, 16-byte aligned, owned by the caller.  Pointers
 *     marked [host] are host pointers read before the call returns.  The library owns only the
 *     context and the scratch memory it allocates inside omnitide_create().
 *   - Counts that one step produces for the next live in device memory (`*_dev` arguments, int32).
 *     A `*_dev` argument may be NULL, in which case the host bound `*_max` is the exact count.
 *     `*_max` always bounds the device value and sizes the launch.
 *   - Tensor layouts (row-major, dense):
 *         Q        [T][h_q][d]          K/V cache  [S][h_kv][d]        O  [T][h_q][d]
 *     One cache *row* = all KV heads of one token = h_kv*d elements.  Query head h reads KV head
 *     h / (h_q / h_kv).  dtype 0 = bf16 storage, 1 = fp32 storage; accumulation is always fp32.
 *   - Unit table: array of omni_unit in logical (time) order, contiguous: units[u+1].start ==
 *     units[u].start + units[u].len, units[0].start == 0; `event` ids are non-decreasing.
 */
#ifndef OMNITIDE_H
#define OMNITIDE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t omni_status;
enum {
    OMNI_OK = 0,
    OMNI_ERR_INVALID_ARG = 1,
    OMNI_ERR_UNSUPPORTED = 2,
    OMNI_ERR_CUDA = 3,
    OMNI_ERR_TIMEOUT = 4,
    OMNI_ERR_CAPACITY = 5
};

/* bits of the device status word (omnitide_poll_status) */
enum {
    OMNI_DEV_TIMEOUT = 1,      /* a bounded on-device wait ran out */
    OMNI_DEV_BAD_UNITS = 2,    /* unit table not contiguous / events decreasing / count above capacity */
    OMNI_DEV_BAD_COUNT = 4     /* a device-side count exceeded its host bound */
};

enum { OMNI_DTYPE_BF16 = 0, OMNI_DTYPE_FP32 = 1 };
enum { OMNI_MOD_VIDEO = 0, OMNI_MOD_AUDIO = 1, OMNI_MOD_TEXT = 2 };
/* retention groups / allocation classes (Section 4 "OmniPick"; Section 6.1 "Placing entries") */
enum { OMNI_GROUP_MUST_KEEP = 0, OMNI_GROUP_SELECTED = 1, OMNI_GROUP_RECENT = 2 };
enum { OMNI_KEEP_DROPPED = 0, OMNI_KEEP_SINK_PREFIX = 1 /* reserved */, OMNI_KEEP_WHOLE = 2 };
enum { OMNI_PAGE_EMPTY = 255 };
enum { OMNI_FLAG_BOUNDARY = 1 };  /* omni_unit.flags bit 0: a boundary span (Section 5.1), kept whole while its event survives */
enum { OMNI_COMPACT_PACK = 0 };

typedef struct {
    int32_t h_q, h_kv, d;
    int32_t dtype;      /* OMNI_DTYPE_* of Q/K/V storage */
    int32_t s_cap;      /* largest history (cache slots) any call will pass */
    int32_t u_cap;      /* largest number of history units */
    int32_t t_cap;      /* largest chunk (tokens) */
} omni_geometry;

/* One typed span of the stream (Section 2.1 "Streaming units"; Section 5.2 unit records). */
typedef struct {
    int32_t start;      /* first token: cache slot (history) or row in the chunk (chunk units) */
    int32_t len;        /* tokens, > 0 */
    int32_t modality;   /* OMNI_MOD_* */
    int32_t event;      /* streaming event the span belongs to */
    int32_t group;      /* OMNI_GROUP_* */
    int32_t flags;      /* bit 0 = OMNI_FLAG_BOUNDARY; the other bits are opaque; carried through */
} omni_unit;

typedef struct {
    int32_t budget;             /* retained-history target in tokens (low watermark, Section 5.1) */
    int32_t n_recent_events;    /* newest events kept whole */
    int32_t modality_cap[3];    /* per-modality token cap on selected (non-protected) units; <0 = none */
} omni_select_params;

/* Parameters of the paper's own score-free retention plan (Section 5.1).  The paper leaves the values open. */
typedef struct {
    int32_t high_watermark;     /* retention starts only when the history exceeds it */
    int32_t low_watermark;      /* trimming target (not a strict bound) */
    int32_t n_recent_events;    /* newest events kept whole */
    int32_t sink_prefix[3];     /* tokens kept at the start of an older image/video or audio span (text entry unused) */
    int32_t text_budget;        /* tokens of older text spans kept, oldest first */
} omni_structural_params;

/* RoPE of the cached keys (Section 5.2 names RoPE only; the rest are the model's parameters). */
typedef struct {
    float theta_base;   /* frequency base, e.g. 10000 or 1000000 */
    int32_t n_dims;     /* rotated dimensions per head: even, <= d; dimension i pairs with i + n_dims / 2 */
} omni_rope_params;

/* Integer results of one compaction, written to device memory. */
typedef struct {
    int32_t n_kept;         /* rows retained */
    int32_t span_pages;     /* ceil(n_kept / page_size): page-rounded physical span (Section 6.2) */
    int32_t rows_moved;     /* retained rows whose slot changed */
    int32_t part_begin[4];  /* first slot of must-keep, selected-history, recent-context, end */
    int32_t reserved;
} omni_compact_info;

/* Allocation classes of Section 6.1, the low two bits of a slot_class byte; bit 7 marks an entry that was
 * retained from a partially evicted unit (a candidate of the class-aware migration, Section 6.2). */
enum {
    OMNI_CLASS_MUST_KEEP = 0,
    OMNI_CLASS_SELECTED = 1,
    OMNI_CLASS_RECENT = 2,
    OMNI_CLASS_CANDIDATE = 0x80
};
#define OMNI_PAGE_MIXED 254   /* page label: live entries of more than one class */
#define OMNI_PAGE_EMPTY 255   /* page label: no live entry */

/* Outcome of omnipage_migrate_class (32 bytes). */
typedef struct omni_class_info {
    int32_t accepted;          /* 1 if the plan reduced the active pages or the active subblocks and was carried out */
    int32_t n_moves;           /* rows moved (0 when rejected) */
    int32_t n_candidates;      /* candidates the planner visited */
    int32_t pages_before, pages_after;          /* pages that hold a live entry */
    int32_t subblocks_before, subblocks_after;  /* subblocks that hold a live entry */
    int32_t reserved;
} omni_class_info;

typedef struct omnitide_ctx omnitide_ctx;

/* Creates a context for one geometry on the current device and allocates its scratch memory.
 * Returns OMNI_ERR_UNSUPPORTED for h_q % h_kv != 0, d not a multiple of 8 or > 256, or a device
 * that is not sm_100; OMNI_ERR_CUDA if an allocation fails.  *ctx_out is NULL on failure. */
omni_status omnitide_create(omnitide_ctx** ctx_out, const omni_geometry* geometry /*[host]*/);
omni_status omnitide_destroy(omnitide_ctx* ctx);

/* Copies the device status word (OMNI_DEV_* bits, 0 = clean) to *device_status_out [host] and
 * clears it.  Synchronises `stream` first. */
omni_status omnitide_poll_status(omnitide_ctx* ctx, void* stream, int32_t* device_status_out);

/* Text of the last host-side error on this context (static storage inside the context). */
const char* omnitide_last_error(const omnitide_ctx* ctx);

/*
 * (a1) Unit scoring.  For every history unit u:
 *      s_hij  = scale * <Q[i][h], K[j][h / G]>                 i < t, j < n_hist
 *      a_hij  = softmax over the n_hist history keys of s_hij   (chunk keys excluded)
 *      mass_u = (1 / (h_q * t)) * sum over h, i and j in u of a_hij
 *      score_u = w_modality[modality_u] * mass_u * n_hist / len_u
 * This is the per-span averaged attention weight that the paper's design study measures offline
 * (Section 5, "Key insight"), weighted per modality ("Modality-asymmetric attention"); the paper's
 * own OmniPick is score-free, so the formula is this library's reading, not the paper's.
 *   q [dev] t*h_q*d, k_cache [dev] rows 0..n_hist-1 used, units [dev] n_units entries,
 *   w_modality [host] 3 floats, scale <= 0 means 1/sqrt(d),
 *   scores_out [dev] n_units_max floats, mass_out [dev] nullable.
 * The QK^T contraction runs on tcgen05 tensor cores for bf16 with d == 128, on CUDA cores otherwise.
 */
omni_status omnitide_score_units(omnitide_ctx* ctx, void* stream,
                                 const void* q, int32_t t,
                                 const void* k_cache, const int32_t* n_hist_dev, int32_t n_hist_max,
                                 const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                 const float* w_modality, float scale,
                                 float* scores_out, float* mass_out);

/*
 * (a2) Budgeted unit selection (Section 5.1 for what the paper fixes: protected prefix, newest
 * events kept whole, spans never cut at a token position, the budget a trimming target).
 *   1. protected = units of group must-keep, plus every unit of the n_recent_events newest events;
 *   2. if the protected tokens already reach the budget, exactly the protected set is kept;
 *   3. otherwise the other units are visited by descending score (ties: later unit first, NaN last)
 *      and one is taken iff it fits the remaining budget and its modality's remaining cap;
 *   4. survivors are re-indexed (Section 5.2): units_out holds the kept units in order with `start`
 *      = kept tokens before them, modality/event/flags preserved, group = must-keep if it was,
 *      else recent-context if in a newest event, else selected-history.
 * Outputs [dev]: unit_keep_out[n_units] (OMNI_KEEP_*), keep_mask_out[n_hist] (1 = retained),
 * n_kept_out, units_out (capacity n_units_max), n_units_out.
 */
omni_status omnitide_select_units(omnitide_ctx* ctx, void* stream,
                                  const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                  const float* scores, const omni_select_params* params /*[host]*/,
                                  uint8_t* unit_keep_out, uint8_t* keep_mask_out, int32_t n_hist_max,
                                  int32_t* n_kept_out, omni_unit* units_out, int32_t* n_units_out);

/*
 * (next row: OmniPick as the paper describes it, Section 5.1 "Structure-aware retention planning") Score-free
 * retention plan from unit metadata alone.  An event (the paper's "unit") is the run of spans that share an
 * event id.
 *   0. nothing happens unless the history exceeds high_watermark;
 *   1. must-keep spans and the n_recent_events newest events are kept whole;
 *   2. older events, oldest to newest: a boundary span (OMNI_FLAG_BOUNDARY) is kept whole, an image/video or
 *      audio span keeps its first sink_prefix[modality] tokens, text spans are kept whole, oldest first, until
 *      text_budget is exhausted (the first one that does not fit ends it);
 *   3. while the plan still exceeds low_watermark, whole events are dropped oldest first, partially retained
 *      events before complete ones, until the target is met or one event remains;
 *   4. survivors are re-indexed (Section 5.2) as in omnitide_select_units; a shortened span keeps its record
 *      with the new length.
 * Outputs [dev]: unit_keep_out[n_units] (0 dropped, 1 sink prefix only, 2 whole), unit_kept_len_out[n_units]
 * (nullable), keep_mask_out[n_hist] (nullable, 16-byte aligned), n_kept_out, units_out, n_units_out.
 * Together with omnipage_compact_units(..., unit_kept_len, ...) this is the path with no scoring at all.
 */
omni_status omnitide_plan_structural(omnitide_ctx* ctx, void* stream,
                                     const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                     const omni_structural_params* params /*[host]*/,
                                     uint8_t* unit_keep_out, int32_t* unit_kept_len_out, uint8_t* keep_mask_out,
                                     int32_t n_hist_max, int32_t* n_kept_out, omni_unit* units_out, int32_t* n_units_out);

/*
 * (a3) OmniPage eager compaction (Section 6, "Compaction-movement trade-off": pack every retained
 * entry into a contiguous prefix; Section 6.1 for allocation classes and page promotion; Section 6.2
 * for the page-rounded span and for copy semantics: reads of all sources precede all writes).
 *   for s in [0, s_span): if keep_mask[s]: slot_map[s] = n; dst[n] = src[s]; n++   else slot_map[s] = -1
 * Rows are copied bit for bit.  k_dst/v_dst may be different buffers (one read + one write per row,
 * no staging) or equal to k_src/v_src (in place: rows are staged through context scratch).
 * Because units are in time order and group rank grows with recency, the stable pack is already the
 * retention-partitioned order must-keep | selected-history | recent-context; part_begin reports the
 * partition starts from units_kept (the table omnitide_select_units wrote; may be NULL).
 * page_class_out[p] for p < ceil(s_span_max / page_size): 0 if page p holds a must-keep row, else 1 if
 * it holds page_size retained rows (promoted to selected-history), else 2 if partly filled (stays
 * recent-context), else OMNI_PAGE_EMPTY.
 *   slot_map_out [dev] s_span_max int32 (nullable), info_out [dev], page_class_out [dev] nullable.
 *   keep_mask [dev] is read in aligned 16-byte vectors: the buffer must extend to s_span_max rounded up to a
 *   multiple of 16 bytes; bytes at and beyond *s_span_dev are ignored.  Calls on one context must not overlap
 *   (the CTAs of the kernel exchange their counts through context scratch).
 * mode must be OMNI_COMPACT_PACK.
 */
omni_status omnipage_compact(omnitide_ctx* ctx, void* stream,
                             const void* k_src, const void* v_src, void* k_dst, void* v_dst,
                             const uint8_t* keep_mask, const int32_t* s_span_dev, int32_t s_span_max,
                             int32_t page_size, int32_t mode,
                             const omni_unit* units_kept, const int32_t* n_units_kept_dev, int32_t n_units_max,
                             int32_t* slot_map_out, omni_compact_info* info_out, uint8_t* page_class_out);

/*
 * (a3, unit-granular form) The same eager pack when the keep decision is one code per UNIT, which is what
 * omnitide_select_units produces (Section 5.1: spans are never cut at a token position; Section 5.2: the unit
 * records carry the layout).  Equivalent to omnipage_compact with
 *   keep_mask[s] = (unit_keep[unit that holds s] != OMNI_KEEP_DROPPED),   s_span = end of the last unit,
 * but no mask is read: the gather is a list of at most n_units contiguous runs, so no CTA has to wait for
 * another one's count and the kernel starts copying after one round trip to the unit table.
 *   units [dev] the history unit table (contiguous, in order), n_units_dev [dev, nullable] / n_units_max [host];
 *   unit_keep [dev] n_units_max bytes (OMNI_KEEP_*); unit_kept_len [dev, nullable] n_units_max int32: the number of
 *   tokens kept at the START of every unit (sink prefixes of omnitide_plan_structural; NULL = kept units are whole);
 *   s_span_max [host] bound on the history length;
 *   units_kept / n_units_kept_dev: the re-indexed table of the survivors (for part_begin; nullable);
 *   slot_map_out [dev] s_span_max int32 (nullable), info_out [dev], page_class_out [dev] nullable, as above.
 * A unit that reaches outside [0, s_span_max) sets OMNI_DEV_BAD_UNITS and is treated as dropped.
 */
omni_status omnipage_compact_units(omnitide_ctx* ctx, void* stream,
                                   const void* k_src, const void* v_src, void* k_dst, void* v_dst,
                                   const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                   const uint8_t* unit_keep, const int32_t* unit_kept_len,
                                   int32_t s_span_max, int32_t page_size,
                                   const omni_unit* units_kept, const int32_t* n_units_kept_dev,
                                   int32_t* slot_map_out, omni_compact_info* info_out, uint8_t* page_class_out);

/*
 * (next row: selective migration, ordered-suffix mode; Section 6.2 "Checking layout improvement")  The mode the paper
 * uses on CUDA, where attention traverses the physical span: scan backward from the end of the span for the smallest
 * page-aligned suffix whose packing shortens the page-rounded span by at least min_pages_saved pages; pack only the
 * live rows of that suffix, in order, to its start; every slot before it keeps its content and its holes.  If no
 * suffix qualifies nothing moves.  In place (moves go through context scratch: reads of all sources precede all
 * writes).  keep_mask [dev, in/out] and *s_span_dev [dev, in/out] describe the layout before and after; the result is
 * what omnitide_chunk_attention_masked takes.  slot_map_out [dev, nullable] s_span_max int32: new slot of every live
 * row, -1 for dead ones.  info_out [dev, nullable]: n_kept = live rows, span_pages = pages of the new span,
 * rows_moved, part_begin = {suffix start or -1, new span, pages saved, old span}.  page_size a multiple of 16.
 */
omni_status omnipage_migrate_suffix(omnitide_ctx* ctx, void* stream, void* k_cache, void* v_cache,
                                    uint8_t* keep_mask, int32_t* s_span_dev, int32_t s_span_max,
                                    int32_t page_size, int32_t min_pages_saved,
                                    int32_t* slot_map_out, omni_compact_info* info_out);

/*
 * (next row: selective migration, class-aware mode; Section 6.2 "Packing scattered entries" and "Checking layout
 * improvement", classes and promotion of Section 6.1)  Plans, checks and carries out the moves that fill earlier
 * holes with the entries retained from partially evicted units.
 *   keep_mask [dev, in/out] s_span_max bytes, 1 = live; slot_class [dev, in/out] s_span_max bytes, read where live:
 *   class in bits 0-1 (OMNI_CLASS_*; the value 3 sets OMNI_DEV_BAD_UNITS and nothing moves), candidate mark in bit 7.
 *   *s_span_dev [dev, nullable] / s_span_max [host]: the span; pages are page_size slots, subblocks `subblock` slots
 *   (subblock divides page_size).
 * Plan: the candidates (live, marked, in a page that is not full) are visited in ascending slot order; a candidate
 * of class c at slot s goes to the smallest slot d < s that is empty in the layout as simulated so far (vacated
 * slots count) and whose page is empty or holds class c only; if there is none it stays.  Nothing else moves.
 * Accept test: the plan is carried out iff it lowers the number of pages, or of subblocks, that hold a live entry.
 * If carried out: K/V rows move in place (all sources are read into context scratch before any destination is
 * written), keep_mask and slot_class follow the entries (vacated slots become 0), and if `promote` is non-zero every
 * page that is now full of selected-history / recent-context entries is relabelled selected-history.
 *   moves_out [dev, nullable] 2 * s_span_max int32: the (source, destination) pairs in plan order, for the caller's
 *   own per-slot metadata; page_class_out [dev, nullable] ceil(s_span_max / page_size) bytes: class of the page's
 *   entries, OMNI_PAGE_MIXED or OMNI_PAGE_EMPTY (pages past the span are not written); info_out [dev] the counts.
 * The layout (one bit per slot, eight bytes per page) must fit one CTA's shared memory, else OMNI_ERR_CAPACITY.
 * The result is a layout for omnitide_chunk_attention_masked.
 */
omni_status omnipage_migrate_class(omnitide_ctx* ctx, void* stream, void* k_cache, void* v_cache,
                                   uint8_t* keep_mask, uint8_t* slot_class, const int32_t* s_span_dev,
                                   int32_t s_span_max, int32_t page_size, int32_t subblock, int32_t promote,
                                   int32_t* moves_out, uint8_t* page_class_out, omni_class_info* info_out);


/*
 * (next row: RoPE position re-index fused into the gather; Section 5.2 "the runtime applies the corresponding RoPE
 * adjustment to cached keys")  omnipage_compact_units with every moved K row re-rotated to its new position while it
 * passes through shared memory.  Positions are slot indices (the cache is dense before and after the pack), so the
 * shift of a row is (destination slot - source slot) <= 0; angle = shift * theta_base^(-2i / n_dims) for the pair
 * (i, i + n_dims/2) of every head; angles in double, rotation in fp32, result rounded to bf16 (nearest even).
 * V rows and all integer outputs are those of omnipage_compact_units.  bf16 caches only.
 */
omni_status omnipage_compact_units_rope(omnitide_ctx* ctx, void* stream,
                                        const void* k_src, const void* v_src, void* k_dst, void* v_dst,
                                        const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                        const uint8_t* unit_keep, const int32_t* unit_kept_len,
                                        int32_t s_span_max, int32_t page_size,
                                        const omni_unit* units_kept, const int32_t* n_units_kept_dev,
                                        int32_t* slot_map_out, omni_compact_info* info_out, uint8_t* page_class_out,
                                        const omni_rope_params* rope /*[host]*/);

/*
 * (next row: cross-layer batching) The unit-granular pack applied to n_layers caches in ONE launch with one shared
 * source -> destination map (Section 6.2 "Executing accepted moves": the mapping is planned once from metadata and
 * every layer's K and V rows follow it).  k_src / v_src / k_dst / v_dst [dev] are device arrays of n_layers
 * device pointers (caller-owned; out of place only: no k_dst[l] may overlap any source).  All other arguments
 * and all outputs are those of omnipage_compact_units (the integer outputs describe the shared map once).
 * Turns the launch-bound single-layer copy into one bandwidth-bound launch.  2 * s_span_max * n_layers < 2^31.
 */
omni_status omnipage_compact_units_batched(omnitide_ctx* ctx, void* stream,
                                           const void* const* k_src, const void* const* v_src,
                                           void* const* k_dst, void* const* v_dst, int32_t n_layers,
                                           const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                           const uint8_t* unit_keep, const int32_t* unit_kept_len,
                                           int32_t s_span_max, int32_t page_size,
                                           const omni_unit* units_kept, const int32_t* n_units_kept_dev,
                                           int32_t* slot_map_out, omni_compact_info* info_out, uint8_t* page_class_out);

/*
 * (a5) Append: new entries enter the recent-context class behind the retained history
 * (Section 6.1).  Copies the chunk's t K/V rows to cache slots [n_kept, n_kept + t), appends the
 * chunk's units to `units` with start += n_kept and group = recent-context, and writes
 * *n_hist_out = n_kept + t, *n_units_out = n_units + n_chunk_units.
 *   n_kept_dev, n_units_dev [dev] in; chunk_units [dev]; n_hist_out / n_units_out [dev] may alias
 *   the inputs.  s_cap / u_cap overflow sets OMNI_DEV_BAD_COUNT and copies nothing.
 */
omni_status omnipage_append(omnitide_ctx* ctx, void* stream,
                            void* k_cache, void* v_cache, const int32_t* n_kept_dev,
                            const void* k_chunk, const void* v_chunk, int32_t t,
                            omni_unit* units, const int32_t* n_units_dev,
                            const omni_unit* chunk_units, int32_t n_chunk_units,
                            int32_t* n_hist_out, int32_t* n_units_out);

/*
 * (a4) GQA chunk-prefill attention (Section 2.1 prefill; Section 3 "Dense attention"):
 *      O[i][h] = sum_j softmax_j(scale * <Q[i][h], k_j>) v_j
 * over j in history rows [0, n_hist) followed by chunk rows [0, i] (causal inside the chunk,
 * diagonal included).  k_chunk/v_chunk may point into the cache behind the history.
 *   o_out [dev] t*h_q*d of out_dtype (OMNI_DTYPE_*), lse_out [dev] t*h_q floats, nullable
 *   (natural-log sum of exponentials of the scaled logits).
 * bf16 with d == 128 runs on tcgen05 tensor cores (TMA-fed, TMEM accumulators); other geometries
 * run on CUDA cores in fp32.
 */
omni_status omnitide_chunk_attention(omnitide_ctx* ctx, void* stream,
                                     const void* q, int32_t t,
                                     const void* k_hist, const void* v_hist,
                                     const int32_t* n_hist_dev, int32_t n_hist_max,
                                     const void* k_chunk, const void* v_chunk,
                                     float scale, void* o_out, int32_t out_dtype, float* lse_out);

/*
 * One whole pass (a1..a5 in order) for one layer with every tensor resident on the device.
 * State in: k_cache/v_cache rows [0, *n_hist_dev), units[0, *n_units_dev).  State out: the compacted
 * history plus the chunk in k_cache_out/v_cache_out (must be different buffers), units_out, and the
 * updated counts in n_hist_out / n_units_out.  Work buffers for scores, masks and the slot map come
 * from the context.  o_out as in omnitide_chunk_attention; info_out nullable.
 */
omni_status omnitide_chunk_step(omnitide_ctx* ctx, void* stream,
                                const void* q, const void* k_chunk, const void* v_chunk, int32_t t,
                                const omni_unit* chunk_units, int32_t n_chunk_units,
                                const void* k_cache, const void* v_cache,
                                const int32_t* n_hist_dev, int32_t n_hist_max,
                                const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                const float* w_modality, const omni_select_params* params, int32_t page_size,
                                float scale,
                                void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                int32_t* n_hist_out, int32_t* n_units_out,
                                void* o_out, int32_t out_dtype, omni_compact_info* info_out);

/*
 * (next row: layouts with holes)  omnitide_chunk_attention over a history in which only the slots marked in
 * hist_keep_mask are live (Section 6, "Fragmentation after logical eviction": logical deletion leaves masked holes
 * between surviving entries; Section 6.1: a tile is skipped only when all its entries are masked).  The span
 * [0, *s_span_dev) of k_hist / v_hist is presented; 128-key blocks with no live slot are skipped (no load, no MMA),
 * the other blocks have their dead columns masked.  Equals attention over the live rows in order.
 *   hist_keep_mask [dev] s_span_max bytes readable up to a multiple of 16 (nonzero = live), 16-byte aligned;
 *   dead slots inside the span must hold finite values (evicted entries do); slots beyond the span may hold anything.
 */
omni_status omnitide_chunk_attention_masked(omnitide_ctx* ctx, void* stream,
                                            const void* q, int32_t t,
                                            const void* k_hist, const void* v_hist, const uint8_t* hist_keep_mask,
                                            const int32_t* s_span_dev, int32_t s_span_max,
                                            const void* k_chunk, const void* v_chunk, float scale,
                                            void* o_out, int32_t out_dtype, float* lse_out);

/*
 * The pass as the paper runs it (no scoring): omnitide_plan_structural -> omnipage_compact_units with the planned
 * prefix lengths -> omnitide_chunk_attention -> omnipage_append.  Arguments as omnitide_chunk_step, with the
 * structural parameters in place of the modality weights and the selection parameters.
 */
omni_status omnitide_chunk_step_structural(omnitide_ctx* ctx, void* stream,
                                           const void* q, const void* k_chunk, const void* v_chunk, int32_t t,
                                           const omni_unit* chunk_units, int32_t n_chunk_units,
                                           const void* k_cache, const void* v_cache,
                                           const int32_t* n_hist_dev, int32_t n_hist_max,
                                           const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                           const omni_structural_params* params /*[host]*/, int32_t page_size, float scale,
                                           void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                           int32_t* n_hist_out, int32_t* n_units_out,
                                           void* o_out, int32_t out_dtype, omni_compact_info* info_out);

/*
 * The same pass for a caller whose chunk lives in host memory: q/k_chunk/v_chunk/chunk_units are
 * HOST pointers (pinned memory recommended) copied to context staging buffers on `stream`, and the
 * attention output is copied back to o_host (out_dtype elements).  The call returns after the
 * copies and kernels are enqueued; synchronise the stream before reading o_host.
 */
omni_status omnitide_chunk_step_host(omnitide_ctx* ctx, void* stream,
                                     const void* q_host, const void* k_chunk_host, const void* v_chunk_host, int32_t t,
                                     const omni_unit* chunk_units_host, int32_t n_chunk_units,
                                     const void* k_cache, const void* v_cache,
                                     const int32_t* n_hist_dev, int32_t n_hist_max,
                                     const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                     const float* w_modality, const omni_select_params* params, int32_t page_size,
                                     float scale,
                                     void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                     int32_t* n_hist_out, int32_t* n_units_out,
                                     void* o_host, int32_t out_dtype, omni_compact_info* info_out);

/*
 * The same pass for a caller that streams chunks: the call only enqueues.  The context keeps two sets of staging
 * buffers and runs the uploads of call n on a copy stream under the kernels of call n - 1, and the download of
 * call n on a second copy stream under the kernels of call n + 1; the kernels themselves run on `stream` in call
 * order (call n + 1 reads the cache state call n wrote).  Arguments as omnitide_chunk_step_host.
 * The host input buffers of a call may be rewritten, and o_host read, only after omnitide_host_wait (or a
 * synchronisation of the whole device); pinned host memory is needed for the copies to overlap.  Staging is
 * allocated on the first call (synchronously).
 */
omni_status omnitide_chunk_step_host_pipelined(omnitide_ctx* ctx, void* stream,
                                               const void* q_host, const void* k_chunk_host, const void* v_chunk_host,
                                               int32_t t, const omni_unit* chunk_units_host, int32_t n_chunk_units,
                                               const void* k_cache, const void* v_cache,
                                               const int32_t* n_hist_dev, int32_t n_hist_max,
                                               const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                               const float* w_modality, const omni_select_params* params,
                                               int32_t page_size, float scale,
                                               void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                               int32_t* n_hist_out, int32_t* n_units_out,
                                               void* o_host, int32_t out_dtype, omni_compact_info* info_out);

/* Blocks until every upload and download enqueued by the host entry points of this context has completed
 * (the kernels on the caller's stream are the caller's to synchronise). */
omni_status omnitide_host_wait(omnitide_ctx* ctx);

/*
 * Unit scoring for callers that cannot allocate.  (The paper has no counterpart: this is a
 * packaging variant of omnitide_score_units, same formula, computed by the fp32 CUDA-core kernel.)
 *
 * Some hosts of this library may not call cudaMalloc at all: a serving runtime that hands every
 * byte of HBM to its own KV-cache pool at start-up, so that a later cudaMalloc fails or takes memory
 * the pool believes it owns; or a latency-critical loop in which cudaMalloc/cudaFree, which
 * synchronise the whole device, would stall every other stream.  Such callers cannot create an
 * omnitide_ctx (creation allocates scratch).  This entry point needs no context and allocates
 * nothing: the per-unit accumulators it needs live in a fixed array of
 * OMNITIDE_NOALLOC_MAX_UNITS doubles (8 KiB) inside the library's device image, present on every
 * GPU that loads the library until the process exits.
 *
 *   - n_units above OMNITIDE_NOALLOC_MAX_UNITS is refused with OMNI_ERR_CAPACITY (nothing is launched).
 *   - Counts are host values here (n_hist, n_units); q, k_cache, units, scores_out, mass_out are
 *     device pointers owned by the caller as in omnitide_score_units; mass_out may be NULL.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current); make that first call outside any stream capture.
 *   - Every call on a device shares the one array.  The call clears the accumulators it uses before
 *     adding into them, so back-to-back calls on one stream are independent; two calls whose kernels
 *     can overlap on the GPU (different streams, no ordering between them) race on the array and
 *     must be serialised by the caller.
 */
#define OMNITIDE_NOALLOC_MAX_UNITS 1024
omni_status omnitide_score_units_noalloc(void* stream, int32_t h_q, int32_t h_kv, int32_t d, int32_t dtype,
                                         const void* q, int32_t t, const void* k_cache, int32_t n_hist,
                                         const omni_unit* units, int32_t n_units,
                                         const float* w_modality, float scale,
                                         float* scores_out, float* mass_out);

/* Options.  OMNI_OPT_FORCE_CUDA_CORES != 0 routes scoring and attention through the fp32 CUDA-core
 * kernels even where the tensor-core kernels apply (a second implementation for cross-checks).
 * OMNI_OPT_SCORE_WINDOW = W > 0 makes omnitide_chunk_step (and its host form) score the history with the last W
 * queries of the chunk only, a trailing observation window as in the score-based methods the paper cites (Section 3);
 * 0 (default) scores with every query.  A caller of omnitide_score_units gets the same by passing that row range.
 * OMNI_OPT_HIGH_WATERMARK = H > 0 gives omnitide_chunk_step (and its host forms) the paper's hysteresis (Section 5.1:
 * retention starts only above a high watermark and trims to the low one, here the selection budget): a call whose
 * n_hist_max is at most H launches no scoring kernel and keeps every unit (the history is copied whole to the output
 * cache); a call whose bound exceeds H runs the full pass.  The decision is the host's, from the bound it was given,
 * so a caller that wants rounds to be rare passes a tight n_hist_max.  0 (default): every call runs the full pass.
 * (Scoring only every k-th chunk is the same mechanism driven by the caller: a watermark of INT32_MAX on the other
 * chunks, the real one, or 0, on every k-th.) */
enum { OMNI_OPT_FORCE_CUDA_CORES = 1, OMNI_OPT_SCORE_WINDOW = 2, OMNI_OPT_HIGH_WATERMARK = 3 };
omni_status omnitide_set_option(omnitide_ctx* ctx, int32_t option, int32_t value);

/* Number of kernels this library has launched on this context since creation (for accounting). */
int64_t omnitide_launch_count(const omnitide_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* OMNITIDE_H */
