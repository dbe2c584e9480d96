/*
 * wnw.h -- C ABI of the WnW decode hot path for NVIDIA B200 (sm_100a).
 *
 * WnW (Waxing-and-Waning KV cache) serves long-form speech LLM decoding with a
 * GQA KV cache whose audio KV-heads carry offline-assigned roles (Method
 * section, "Method Overview" and "Three-Way Classification"):
 *   anchor  heads keep all audio KV on the GPU; their decode-time softmax
 *           weights are the importance signal (Eq. 2);
 *   tidal   heads keep a budgeted set of audio chunks on the GPU and the rest
 *           in pinned host memory, recalled on demand ("Dynamic Chunk
 *           Selection");
 *   fixed   heads keep a static subset chosen at prefill ("Prefill
 *           Compression"); the rest is discarded.
 * Text KV (prompt and generated tokens) is always kept in full.
 *
 * This library implements the per-token, per-layer decode step in the
 * chunk-granular form: non-overlapping chunks of `chunk_tokens` audio tokens
 * are the unit of scoring, selection, residency and transfer; each non-anchor
 * head keeps S = min(C, max(1, floor((double)budget * C + 1e-6))) chunks of the
 * C = ceil(T_a / chunk_tokens) chunks of a sequence.
 *
 * Conventions
 *   - All tensor arguments named *_dev are DEVICE pointers to bf16 data
 *     (2 bytes per element, row-major, innermost index last), 16-byte aligned.
 *     Arguments named *_host are HOST pointers.  The library never takes
 *     ownership of caller buffers; they must stay valid until the work queued
 *     on the given stream has completed.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Every call returns a wnw_status_t and never throws or aborts.  On error,
 *     out-parameters are left untouched.  Errors detected on the device
 *     (table invariant violations) are sticky and reported by wnw_sync.
 *   - A cache object is not thread-safe.  Calls for one cache must come from
 *     one thread at a time.
 *   - Position encoding (RoPE) is the caller's job: q and K arrive rotated.
 */
#ifndef WNW_H_
#define WNW_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wnw_cache wnw_cache_t; /* opaque, library-owned */

typedef enum {
  WNW_OK = 0,
  WNW_ERR_INVALID_ARG = 1,
  WNW_ERR_STATE = 2,      /* call out of order (decode before prefill, layer order, ...) */
  WNW_ERR_OOM_DEVICE = 3,
  WNW_ERR_OOM_HOST = 4,   /* pinned host allocation failed */
  WNW_ERR_CUDA = 5,       /* a CUDA runtime call failed */
  WNW_ERR_CAPACITY = 6,   /* text or audio capacity exceeded */
  WNW_ERR_TIMEOUT = 7,    /* a bounded device-side wait ran out (sticky, reported by wnw_sync); the context stays usable */
  WNW_ERR_UNSUPPORTED = 8,/* shape outside what the kernels are built for */
  WNW_ERR_DEVICE_CHECK = 9/* a device-side consistency check failed (sticky) */
} wnw_status_t;

enum { WNW_ROLE_ANCHOR = 0, WNW_ROLE_TIDAL = 1, WNW_ROLE_FIXED = 2 };

/* Storage mode.  TIERED is WnW.  FULL stores every head in full on the GPU
 * (the "Full Cache" baseline of the Baselines paragraph) and serves
 * wnw_decode_layer_full; roles are ignored for storage in that mode. */
enum { WNW_MODE_TIERED = 0, WNW_MODE_FULL = 1 };

/* Which anchor heads rank a tidal layer's chunks.
 *   PER_LAYER  the layer's own anchor heads, else those of the nearest layer that has some (ties to the lower layer)
 *   GLOBAL     Eq. 2 as printed: one accumulator over ALL anchor (layer, q-head) pairs of the step, added in layer
 *              order; every tidal layer takes the same selection, made once the last layer of the step has run */
enum { WNW_SCOPE_PER_LAYER = 0, WNW_SCOPE_GLOBAL = 1 };

/* How the tidal tables evolve ("Chunk Structure", "Dynamic Chunk Selection").
 *   HARD_BUDGET  a fixed pool of S = max(1, floor(budget*C)) slots per (sequence, layer); non-overlapping chunks of
 *                chunk_tokens; a miss takes a free slot, else evicts the least recently selected chunk that is not
 *                selected now.  evict_lag is not used.
 *   SEGMENT_LAG  the paper's form: chunk_tokens is the SEGMENT length n_s; a chunk is two consecutive segments, so
 *                adjacent chunks share one (chunk j = segments j, j+1; ranked by the mean over its tokens; wnw_get_selected
 *                returns chunk indices).  The S_base = max(1, floor(budget*C)) segments placed at prefill stay resident
 *                for good; the missing segments of the selected chunks are fetched into 2*topk*(evict_lag+1) further
 *                slots (never short), and a fetched segment left unselected for evict_lag consecutive steps is dropped
 *                (its host copy persists).  Fixed heads keep S_base segments.  wnw_get_seq_dims reports all slots;
 *                wnw_get_base_slots the permanent ones.
 *   SEGMENT_LAG_TOKEN_BASE  SEGMENT_LAG with the permanent base kept token by token ("Prefill Compression" as printed):
 *                no segment is permanent as a whole (wnw_get_base_slots = 0; a table has only the 2*topk*(evict_lag+1)
 *                dynamic slots).  Every tidal head keeps for good, in a compact store of its own, its best
 *                floor(retention*length) positions of every segment (by its own prefill score); the host mirror holds
 *                each segment with the positions that are NOT in the base first, so a fetched segment contributes
 *                exactly its complement.  A tidal head attends to [text | its kept positions | the complements of the
 *                segments in the layer's dynamic slots].  Sequences must be placed with wnw_place_prefill_tokens
 *                (segment_tokens = chunk_tokens); wnw_place_prefill and _multi return WNW_ERR_STATE.
 *                A compact store holds floor(budget*C)+2*topk*(evict_lag+1) blocks of chunk_tokens positions. */
enum { WNW_RESIDENCY_HARD_BUDGET = 0, WNW_RESIDENCY_SEGMENT_LAG = 1, WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE = 2 };

/* How recall copies are issued (for measurement; results are identical for 0 and 1):
 *   0  side stream, overlapped with the following layers (default)
 *   1  on the caller's stream right after the layer (the paper's naive schedule, Limitations section)
 *   2  skipped: tables update, no bytes move (timing experiments only; outputs become wrong) */
enum { WNW_RECALL_SIDE_STREAM = 0, WNW_RECALL_INLINE = 1, WNW_RECALL_SKIP = 2 };

/* Storage format of the tidal tier: the audio K,V of tidal heads in the pinned host mirror and in the GPU slot pool
 * (KV quantisation is orthogonal to the method: Baselines paragraph, footnote on KV quantisation).
 *   BF16      as given (default)
 *   FP8_E4M3  one byte per element: e4m3 (4 exponent bits, bias 7, 3 mantissa bits, subnormals, largest finite 448) with
 *             one power-of-two scale 2^e per (chunk, tidal head, K|V), e the integer with max|x| / 2^e in (224, 448]
 *             (0 for an all-zero block); elements are x / 2^e rounded to nearest, ties to even.  Host-link bytes per
 *             recalled chunk and the HBM bytes tidal heads read both halve.  The stored value of an element, e4m3 * 2^e,
 *             is an exact bf16 number, and EVERYTHING the library computes for a tidal head (prefill scores included)
 *             uses stored values, so results agree, within the tolerances stated for outputs and scores, with those of a
 *             BF16 cache given the stored values as input (the two products with an e4m3 block take the query and the
 *             softmax weights as fp16: exact for query elements inside fp16's normal range; |q| > 65504 is not supported
 *             with this format).  Text rows, anchor heads and fixed heads stay bf16.  Needs head_dim 128, a residency other than SEGMENT_LAG_TOKEN_BASE
 *             and streaming_audio = 0 (a growing chunk would have to be re-scaled): WNW_ERR_UNSUPPORTED otherwise.
 *             wnw_get_slot_kv returns the stored values as bf16. */
enum { WNW_TIDAL_KV_BF16 = 0, WNW_TIDAL_KV_FP8_E4M3 = 1 };

typedef struct {
  int32_t n_layers, n_q_heads, n_kv_heads; /* n_q_heads % n_kv_heads == 0, group <= 16 */
  int32_t head_dim;                        /* 64 or 128 */
  int32_t max_batch;                       /* sequences the cache can hold */
  int32_t max_audio_tokens;                /* per sequence */
  int32_t max_text_tokens;                 /* per sequence, prompt text + every decode append */
  int32_t chunk_tokens;                    /* n_c >= 1 (e.g. ceil(4 s * 12.5 tok/s) = 50, "Chunk Structure"); stored padded to 16 rows */
  int32_t topk;                            /* k, chunks selected per step; 0 -> 3 (the paper's k) */
  int32_t evict_lag;                       /* the paper's delta: steps a fetched segment may stay unselected before it is released
                                            * (SEGMENT_LAG residencies; HARD_BUDGET evicts the least recently selected chunk instead) */
  float budget;                            /* (0,1]; see S above */
  float softmax_scale;                     /* 0 -> 1/sqrt(head_dim) (Eq. 2) */
  const uint8_t *roles;                    /* HOST [n_layers * n_kv_heads], WNW_ROLE_*, copied */
  int32_t device;                          /* CUDA ordinal */
  int32_t mode;                            /* WNW_MODE_* */
  int32_t recall_mode;                     /* WNW_RECALL_* */
  int32_t score_scope;                     /* WNW_SCOPE_* */
  int32_t residency;                       /* WNW_RESIDENCY_* */
  int32_t defer_selection;                 /* 1: head-sharded serving (see wnw_export_scores): a layer's decode call only adds up the
                                            * chunk scores of the cache's OWN anchor heads; top-k, residency update and recall of every
                                            * tidal layer run in wnw_step_end, on the scores handed back by wnw_import_scores */
  const uint8_t *global_anchor_layers;     /* HOST [n_layers] or NULL, copied.  Head-sharded serving: which layers have an anchor head
                                            * on ANY shard; score routing follows these flags instead of the cache's own roles, and a
                                            * cache may then hold tidal heads without an anchor head of its own */
  int32_t streaming_audio;                 /* 1: clips may grow after placement (wnw_append_audio): every sequence's pinned host
                                            * mirror is sized and laid out for max_audio_tokens.  0: mirrors are sized by the
                                            * placed clip and wnw_append_audio is refused */
  int32_t tidal_kv_format;                 /* WNW_TIDAL_KV_* */
} wnw_config_t;

typedef struct {
  int64_t steps;            /* decode steps completed (sum over sequences) */
  int64_t hits, misses;     /* selected chunks found resident / recalled */
  int64_t evictions;        /* residents displaced */
  int64_t recall_bytes;     /* bytes copied host -> slot pool */
  int64_t resident_audio_tokens; /* audio tokens on the GPU now, all heads (r_GPU numerator, Audio KV retention paragraph) */
  int64_t host_audio_tokens;     /* audio tokens of tidal heads held in host memory and not on the GPU */
  int64_t full_audio_tokens;     /* L * H_kv * T_a summed over placed sequences (denominator) */
} wnw_stats_t;

/* Create a cache: head roles from the offline triage, GPU budget, capacities.
 * Allocates all device stores up front; pinned host mirrors are allocated per
 * sequence at prefill.  Rejects: tidal heads with no anchor anywhere, head_dim
 * not in {64,128}, budget outside (0,1],
 * group > 16.  ("Three-Way Classification"; Eq. 1 budget; "Chunk Structure".) */
wnw_status_t wnw_create(const wnw_config_t *cfg_host, wnw_cache_t **out);

/* Frees everything the cache owns.  Synchronises the device first. */
wnw_status_t wnw_destroy(wnw_cache_t *cache);

/* Place one layer's prefill KV of one sequence ("Prefill Compression", chunk-level).
 *   k_dev, v_dev : [n_tokens][n_kv_heads][head_dim] bf16; tokens [audio_begin, audio_end) are audio,
 *                  all others text, order preserved within each kind.
 *   q_last_dev   : [n_q_heads][head_dim] bf16, the last prefix query; ranks chunks for non-anchor heads:
 *                  pre[c] = sum over the head's query group and tau in c of softmax(q_last K / sqrt d)_tau.
 *                  Fixed head keeps its own top-S chunks; the layer's tidal heads share one table holding the
 *                  top-S chunks of their summed pre (rank r in slot r).  May be NULL if the sequence has no audio
 *                  or in FULL mode.
 * Layers of a sequence must be placed in order 0..n_layers-1 with the same token counts; placing layer 0 again
 * re-initialises the sequence.  Work is queued on cuda_stream; the caller's buffers may be released once that
 * work has completed.  Tidal heads' audio KV is mirrored to pinned host memory allocated here. */
wnw_status_t wnw_place_prefill(wnw_cache_t *cache, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                               int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_last_dev,
                               void *cuda_stream);
/* The same with the prefill score summed over SEVERAL text queries ("Prefill Compression": p_prefill is the attention
 * from the text queries aggregated over them): q_text_dev is [n_queries][n_q_heads][head_dim] bf16, every query
 * attends to the whole prefill key set; one scoring pass per query, added in query order. */
wnw_status_t wnw_place_prefill_multi(wnw_cache_t *cache, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                     int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_text_dev,
                                     int32_t n_queries, void *cuda_stream);
/* Prefill placement with the FIXED heads compressed token by token ("Prefill Compression", per-head retention from
 * Eq. 1).  Anchor heads, tidal tables, slots and host mirrors are placed exactly as by wnw_place_prefill_multi.  Every
 * fixed KV-head h of the layer then keeps, instead of whole chunks, single audio positions:
 *   p[tau]      = sum over the n_queries text queries and the head's q-heads of the softmax weight of audio position tau
 *                 (softmax over the whole prefix, fp32);
 *   variant 0   : inside every segment of segment_tokens positions (the last may be shorter) the
 *                 floor((double)retention[h] * length) positions with the largest p, the earlier position on equal p;
 *   variant 1   : the same number of positions taken from the whole head with no per-segment quota (the paper's
 *                 global top-k ablation of the prefill selection).
 * The kept positions, in ascending order, fill the head's compact store; decode attends to [text | kept positions].
 *   retention   : HOST pointer, [n_kv_heads] floats in [0,1]; entries of heads that are not compressed in this layer
 *                 (anchor heads; tidal heads unless the residency is SEGMENT_LAG_TOKEN_BASE) are ignored.  A head may
 *                 keep at most as many positions as its compact store holds (the slots of a tidal table at
 *                 max_audio_tokens, under the lag residencies the budget's share plus the dynamic slots, times
 *                 chunk_tokens): WNW_ERR_CAPACITY otherwise, nothing placed.
 * With the residency SEGMENT_LAG_TOKEN_BASE the layer's tidal heads are compressed the same way, each by its own
 * scores (their tables start empty); then segment_tokens must equal chunk_tokens (WNW_ERR_UNSUPPORTED otherwise).
 * With variant 1 a head's base holds a different number of positions in every segment; a fetched segment then
 * contributes its length minus that number (kept per head and segment on the device).
 * Scratch and the position lists are allocated by the first call (device memory; not allocation-free).  In FULL mode
 * this is wnw_place_prefill_multi.  Errors as wnw_place_prefill; WNW_ERR_INVALID_ARG for a retention outside [0,1],
 * segment_tokens < 1 or an unknown variant. */
wnw_status_t wnw_place_prefill_tokens(wnw_cache_t *cache, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                      int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_text_dev,
                                      int32_t n_queries, const float *retention, int32_t segment_tokens, int32_t variant,
                                      void *cuda_stream);
/* Eq. 1 on the host: retention[i] = min(s_tilde[i] * lambda, 1) for n heads; s_tilde in [0,1] (the normalised
 * importance of a tidal or fixed head), lambda >= 0.  Host pointers. */
wnw_status_t wnw_retention_schedule(const float *s_tilde, int32_t n, float lambda, float *retention);
/* Introspection of a token placement (host pointers; both wait for queued work).
 * wnw_get_token_scores: p[tau] of a fixed head, [T_a] floats, valid for the (seq, layer) of the most recent
 * wnw_place_prefill_tokens call only (WNW_ERR_STATE otherwise).
 * wnw_get_fixed_tokens: the kept positions of a fixed head in ascending order and their number; WNW_ERR_STATE if the
 * head was placed chunk-wise (then wnw_get_fixed_set applies, which in turn returns WNW_ERR_STATE for a head placed
 * token by token). */
wnw_status_t wnw_get_token_scores(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t kv_head, float *scores,
                                  int32_t capacity);
wnw_status_t wnw_get_fixed_tokens(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t kv_head, int32_t *positions,
                                  int32_t capacity, int32_t *n);

/* Streaming audio: the clip of a placed sequence grows by n_tokens audio positions between decode steps (the
 * Limitations section names streaming as the method's setting; how a growing clip enters the tiers is a reading, stated
 * here).  k_dev, v_dev: [n_tokens][n_kv_heads][head_dim] bf16, the new positions of one layer.  The short last chunk fills
 * up first, then new chunks begin.
 *   anchor heads  keep every new position on the GPU and attend to it from the next step on;
 *   tidal heads   get the new positions in their host mirror; a position that belongs to a chunk resident in the slot
 *                 pool is written to the slot as well (a resident chunk is seen grown), a new chunk stays on the host
 *                 until the anchor heads' scores select it.  The slot count follows the budget on the grown clip,
 *                 S = max(1, floor(budget * C)); the added slots start empty;
 *   fixed heads   keep the subset chosen at placement, which is final: they never see a position that arrived later,
 *                 not even inside a chunk they keep.
 * Layers must be given in order 0..n_layers-1, all with the same n_tokens, outside a step; the grown clip is in force
 * once the last layer has been appended (wnw_step_begin is refused in between).  The first layer's call waits for all
 * queued work of the cache.  Work lists are rebuilt by the next step and a captured step must be captured again.
 * Needs streaming_audio = 1 at creation and the HARD_BUDGET residency (or FULL mode, where every head is stored in
 * full): WNW_ERR_UNSUPPORTED otherwise; WNW_ERR_CAPACITY beyond max_audio_tokens; WNW_ERR_STATE out of order. */
wnw_status_t wnw_append_audio(wnw_cache_t *cache, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                              int32_t n_tokens, void *cuda_stream);

/* Open a decode step for the given sequences (HOST array of distinct sequence ids, all fully placed).
 * The order of active_seqs_host is the batch order of q/k_new/v_new/out in wnw_decode_layer. */
wnw_status_t wnw_step_begin(wnw_cache_t *cache, const int32_t *active_seqs_host, int32_t n_active);

/* One layer of one decode step ("Decode-Step Score Aggregation", "Dynamic Chunk Selection").
 *   q_dev             : [n_active][n_q_heads][head_dim] bf16
 *   k_new_dev,v_new_dev: [n_active][n_kv_heads][head_dim] bf16 of the token being generated, appended to the text
 *                       region before attention; both NULL to attend without appending.  Either every layer of
 *                       a step appends or none does.
 *   out_dev           : [n_active][n_q_heads][head_dim] bf16 attention outputs:
 *                       anchor heads over text + all audio; tidal heads over text + the chunks resident at the end
 *                       of the previous step; fixed heads over text + their prefill subset.
 * Also computed on the device, with no host round trip: this layer's chunk scores
 * score_sum[c] = sum over the layer's anchor q-heads and tau in c of the softmax weight (Eq. 2 summed per chunk);
 * for every tidal layer whose score source is now complete (its own anchors, else the nearest anchor layer, ties
 * to the lower layer) the top-k chunks by mean score (ties to the lower index), the residency table update
 * (hit: refresh; miss: lowest free slot, else least recently selected resident not selected now) and the recall
 * of missing chunks from pinned host memory into the slot pool.  The updated table is used from the next step.
 * Layers must be called in order 0..n_layers-1.  TIERED mode only. */
wnw_status_t wnw_decode_layer(wnw_cache_t *cache, int32_t layer, const void *q_dev, const void *k_new_dev,
                              const void *v_new_dev, void *out_dev, void *cuda_stream);

/* Full-cache comparison path ("Full Cache" baseline): same arguments, every head attends to text + all audio,
 * no scores, no selection.  FULL mode only. */
wnw_status_t wnw_decode_layer_full(wnw_cache_t *cache, int32_t layer, const void *q_dev, const void *k_new_dev,
                                   const void *v_new_dev, void *out_dev, void *cuda_stream);

/* Head-sharded serving (one process per GPU, each holding a cache over its own KV heads; Eq. 2's chunk-score vector is all
 * that crosses heads).  With defer_selection = 1, between the last layer's wnw_decode_layer and wnw_step_end:
 *   wnw_export_scores  copies this cache's partial sums, score_sum[active sequence][layer][chunk] over its own anchor
 *                      heads (zero rows for layers whose anchor heads sit on other shards), into scores_dev, a DEVICE
 *                      buffer of [n_active][n_layers][C_max] floats, C_max = ceil(max_audio_tokens / chunk_tokens);
 *   (the caller adds the buffers of all shards up: one all-reduce(sum) over the ranks, in place, on cuda_stream)
 *   wnw_import_scores  takes the sums back; wnw_step_end then selects, updates the tables and recalls from them.
 * Every shard thus makes the same selection for its own tidal heads.  The same exchange runs once per layer at placement
 * for the tidal tables' initial content, which ranks chunks by the prefill score summed over ALL tidal heads of the layer:
 *   wnw_export_prefill_tidal  after wnw_place_prefill of (seq, layer): this cache's sum over its own tidal heads, [C_max] floats;
 *   wnw_import_prefill_tidal  the sum over all shards: the layer's table is ranked anew from it and its slots are filled
 *                             from the host mirror.
 * Both calls of a pair work on cuda_stream in order; eager steps only (wnw_graph_begin is refused in this mode). */
wnw_status_t wnw_export_scores(wnw_cache_t *cache, void *scores_dev, void *cuda_stream);
wnw_status_t wnw_import_scores(wnw_cache_t *cache, const void *scores_dev, void *cuda_stream);
wnw_status_t wnw_export_prefill_tidal(wnw_cache_t *cache, int32_t seq, int32_t layer, void *sums_dev, void *cuda_stream);
wnw_status_t wnw_import_prefill_tidal(wnw_cache_t *cache, int32_t seq, int32_t layer, const void *sums_dev, void *cuda_stream);

/* Close the step: per-sequence step counters and text lengths advance.  All layers must have been called. */
wnw_status_t wnw_step_end(wnw_cache_t *cache, void *cuda_stream);

/* CUDA-graph replay of a decode step (launch overhead of a whole step collapses into one graph launch).
 * wnw_graph_begin prepares the work lists for the given sequences (HOST array, as in wnw_step_begin) and starts
 * capturing on cuda_stream; the caller then issues ONE ordinary step for those sequences on that stream
 * (wnw_step_begin, wnw_decode_layer[_full] for every layer, wnw_step_end) using buffers it will keep at the same
 * addresses; wnw_graph_end finishes the capture.  Nothing executes during capture and the cache's state does not
 * advance.  Each wnw_graph_launch then runs one step for the captured set of sequences with whatever the buffers
 * hold at that time, and advances the cache exactly like an eager step (text length, step counters).  The capture
 * includes the side-stream selection and recall work and joins it before the step ends.  Eager steps and graph
 * launches may be mixed.  A new capture replaces the previous graph.  Re-placing a sequence or changing the active
 * set requires a new capture.  cuda_stream must not be the default (NULL) stream. */
wnw_status_t wnw_graph_begin(wnw_cache_t *cache, const int32_t *active_seqs_host, int32_t n_active, void *cuda_stream);
wnw_status_t wnw_graph_end(wnw_cache_t *cache, void *cuda_stream);
wnw_status_t wnw_graph_launch(wnw_cache_t *cache, void *cuda_stream);

/* Inspection.  Each call drains the cache's streams first.  Out-buffers are HOST memory owned by the caller.
 *   chunk_scores : score_sum of the last completed step, [C] floats (anchor layers only)
 *   prefill_scores: pre[c] of one non-anchor KV-head, [C] floats
 *   selected     : chunk ids in rank order, up to topk
 *   residency    : slot_chunk[S] (-1 = free) and, if stamp_host != NULL, the recency stamps
 *   fixed_set    : the head's chunk ids in prefill rank order
 *   seq_dims     : T_a, current T_t, C, S of a placed sequence
 *   slot_kv      : the K or V rows of one tidal head in one slot, [chunk_tokens][head_dim] bf16 (which: 0 = K, 1 = V) */
wnw_status_t wnw_get_chunk_scores(wnw_cache_t *cache, int32_t seq, int32_t layer, float *scores_host, int32_t *n_chunks);
wnw_status_t wnw_get_prefill_scores(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t kv_head, float *scores_host,
                                    int32_t *n_chunks);
wnw_status_t wnw_get_selected(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t *sel_host, int32_t *n_sel);
wnw_status_t wnw_get_residency(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t *slot_chunk_host,
                               int64_t *stamp_host, int32_t *n_slots);
wnw_status_t wnw_get_fixed_set(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t kv_head, int32_t *chunks_host,
                               int32_t *n);
wnw_status_t wnw_get_seq_dims(wnw_cache_t *cache, int32_t seq, int32_t *audio_tokens, int32_t *text_tokens,
                              int32_t *n_chunks, int32_t *n_slots);
/* Slots of the sequence's tidal tables that hold the prefill placement (all of them under HARD_BUDGET). */
wnw_status_t wnw_get_base_slots(wnw_cache_t *cache, int32_t seq, int32_t *S_base);
wnw_status_t wnw_get_slot_kv(wnw_cache_t *cache, int32_t seq, int32_t layer, int32_t kv_head, int32_t slot, int32_t which,
                             void *rows_host);
wnw_status_t wnw_get_stats(wnw_cache_t *cache, wnw_stats_t *stats_host);

/* How a layer's attention kernel is ordered against the work that precedes it on the caller's stream.
 *   INDEPENDENT  (default) q/k_new/v_new of every layer of the step exist before the step is issued: consecutive layer
 *                kernels are launched programmatically dependent and may overlap freely (they touch disjoint state).
 *   CHAINED      q/k_new/v_new of a layer are written by the work just before it on the stream (a decoder whose layers
 *                feed one another): the kernel still starts early and queues its K/V cache loads, which do not depend
 *                on that work, but waits for the predecessor to complete before it reads q, k_new or v_new.
 *   SERIAL       plain stream order, no early start.
 *   BATCHED      as INDEPENDENT, and in addition no output of the step is read (by the host or by work queued on the
 *                stream between the layer calls) before the step has ended.  Inside a captured step whose selection
 *                work runs at the end of the step (wnw_graph_begin/end with launches smaller than the machine, recall
 *                not inline; or FULL mode) wnw_decode_layer then only records its arguments and the last layer's call
 *                issues the CTAs of all layers together: one launch, or up to three when the step has tidal heads
 *                (the anchor heads, the fixed heads, then, taking the SMs as those leave, the tidal heads'; the step's
 *                selection runs beside the latter two); elsewhere the mode behaves as INDEPENDENT.
 * Takes effect for layers issued afterwards; a captured step keeps the mode it was captured with.  Not allowed inside
 * a step.  The modes cut the work differently, so outputs agree up to the rounding order of the split merge; selections
 * and tables are the same. */
enum { WNW_LAYERS_INDEPENDENT = 0, WNW_LAYERS_CHAINED = 1, WNW_LAYERS_SERIAL = 2, WNW_LAYERS_BATCHED = 3 };
wnw_status_t wnw_set_layer_dependency(wnw_cache_t *cache, int32_t mode);

/* Kernels this cache has launched on the decode path since creation, replayed captured steps included:
 * counts[0] attention, [1] selection, [2] recall, [3] step-end.  Host counters, no synchronisation. */
wnw_status_t wnw_get_launch_counts(wnw_cache_t *cache, int64_t counts[4]);

/* Drain the caller's stream and the recall stream; returns the sticky asynchronous status. */
wnw_status_t wnw_sync(wnw_cache_t *cache);

/* Full attention of ONE query token over a caller-owned K/V buffer, without any allocation.  (The paper has no
 * counterpart: this is a convenience entry for callers that must not allocate.)
 *
 * Some callers cannot call cudaMalloc where they need attention: a serving loop that has given the whole device
 * to its own pool allocator, or a latency-critical decode thread that cannot afford the device-wide
 * synchronisation cudaMalloc and cudaFree imply.  This entry point calls no cudaMalloc, no cudaFree and no
 * allocating library routine (no device allocation of any kind; on the host it works from the stack); its
 * split-K partials, completion counters and status word live in a fixed array of about 0.8 MB inside
 * the library image, which every GPU that loads the library holds until the process exits.
 *
 *   kv_dev        : DEVICE [n_kv_heads][2][padded_tokens][head_dim] bf16; for each KV head the K rows, then the V
 *                   rows.  Rows in [n_tokens, padded_tokens) are read (whole 16-row tiles are fetched) but never
 *                   contribute: they may hold anything, NaN and Inf included
 *   padded_tokens : row capacity per head, a multiple of 16, >= n_tokens
 *   q_dev         : DEVICE [n_q_heads][head_dim] bf16;  out_dev : DEVICE [n_q_heads][head_dim] bf16
 *   softmax_scale : 0 -> 1/sqrt(head_dim)
 * Result: out = softmax(q K^T * scale) V per query head, the same computation wnw_decode_layer_full performs for
 * one sequence.  Limits (beyond them the call returns WNW_ERR_CAPACITY and does nothing): at most 64 KV heads,
 * 128 query heads, group size 16, 1,048,576 padded tokens; head_dim 64 or 128 (else WNW_ERR_UNSUPPORTED).
 * Each call queues two kernels on cuda_stream: a small one that clears the counters, then the attention kernel.
 *
 * The first call on a device looks up the array's device address and opts the kernels into their shared-memory
 * size; make that first call before any stream capture on that device.  Every call shares the one array, which
 * keeps the previous call's contents (the call clears what must start at zero): two calls whose GPU work overlaps
 * in time - different streams, or different threads - race on it.  Calls on one stream are safe back to back.
 *
 * Every device-side wait of the kernel is bounded.  If one ever runs out (a copy that never lands), the kernel
 * finishes on what it has, the output is incomplete, and a sticky bit is set in the array's status word;
 * wnw_attend_static still returned WNW_OK long before.  wnw_attend_static_status waits for the work queued on
 * cuda_stream, reports whether that happened since it was last asked (timed_out = 1) and clears the bit.  It
 * allocates nothing either. */
wnw_status_t wnw_attend_static(const void *kv_dev, int32_t n_tokens, int32_t padded_tokens, const void *q_dev, void *out_dev,
                               int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float softmax_scale, int32_t device,
                               void *cuda_stream);
wnw_status_t wnw_attend_static_status(int32_t device, void *cuda_stream, int32_t *timed_out_host);

const char *wnw_status_string(wnw_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* WNW_H_ */
