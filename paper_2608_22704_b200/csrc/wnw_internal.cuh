// Internal device-side view of a WnW cache and launch-argument structs shared by the kernels
// and the host runtime.  Nothing here is part of the public ABI (see include/wnw.h).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wnw {

typedef __nv_bfloat16 bf16;

constexpr int GR = 16;        // tokens per granule: one mma k16/n16 tile, the unit of loading and of score partials
constexpr int MAX_TOPK = 8;   // upper bound on config topk
constexpr int MAX_G = 16;     // query heads per KV head handled by one m16 tile
constexpr int MAX_AQ = 128;   // anchor query heads of one layer
constexpr int MAX_UPD_BY_VALUE = 8;  // update-list entries carried in kernel parameters; longer lists read the rest from memory

constexpr int ROLE_ANCHOR = 0, ROLE_TIDAL = 1, ROLE_FIXED = 2;

// device status bits (sticky)
constexpr int STATUS_NO_VICTIM = 1;     // table update found no evictable slot
constexpr int STATUS_BAD_TABLE = 2;     // slot/chunk id out of range
constexpr int STATUS_NONFINITE = 4;     // non-finite chunk score
constexpr int STATUS_TIMEOUT = 8;       // a bounded wait on a TMA barrier gave up

struct WorkItem {  // one CTA of the attention kernel; everything static about it is precomputed on the host
  int32_t i;       // index into the active-sequence list
  int32_t h;       // KV head
  int32_t g0, g1;  // granule range in the head's virtual key space [text capacity | audio]
  int32_t b;       // sequence id
  int32_t role;    // ROLE_* the head plays in this launch
  int32_t ridx;    // index among the heads of that role (anchor-like launches: the KV head)
  int32_t T_a;     // audio tokens of the sequence
  int32_t C, S;    // chunks of the sequence; its PERMANENT slots (tidal slots from S on may be empty)
  int32_t T_hint;  // text rows known to exist when the list was built (a lower bound: text only grows)
  int32_t hd_first, hd_count;  // the work items (= split partials) of this item's head: first (relative to the layer's list), number
};
constexpr int INLINE_ITEMS_MAX = 96;  // launches with at most this many items carry them in kernel parameters
struct InlineItems { WorkItem it[INLINE_ITEMS_MAX]; };
struct HeadItems { int32_t first, count; };  // work items (= split partials) of one (active seq, KV head)

struct LayerInfo {
  int32_t n_anchor, n_tidal, n_fixed;
  int32_t anchor_off;   // anchor heads in earlier layers
  int32_t fixed_off;    // fixed heads in earlier layers
  int32_t tid_prefix;   // tidal heads in earlier layers
  int32_t src;          // layer whose scores rank this layer's chunks, -1 if it has no tidal head
  int32_t upd_first, upd_count;  // range in upd_list: layers whose tables are updated in this layer's tail
  long long pool_off;   // element offset of this layer's slots inside one sequence's pool
};

struct Geometry {
  int32_t L, Hq, Hkv, d, g, nc, gpc, topk;  // nc: audio tokens per chunk; gpc: 16-token granules per stored chunk
  int32_t ncp;                              // rows a chunk occupies in every store: nc rounded up to whole granules
  int32_t T_cap_pad, n_tg;         // text capacity (multiple of 16) and its granules
  int32_t C_max, S_max, T_a_pad;   // chunk / slot capacity per sequence; audio capacity padded to whole chunks
  int32_t A_tot, F_tot;            // anchor heads / heads with a compact store per sequence over all layers
  int32_t F_fix;                   // of those, the fixed heads (they come first); the rest are tidal heads' token bases
  int32_t FB;                      // blocks of chunk_tokens rows a compact store holds
  int32_t token_base;              // SEGMENT_LAG with a token-granular permanent base (no permanent slots)
  int32_t lag_mode, delta, plan_cap;  // SEGMENT_LAG residency; its eviction lag; plan entries per (sequence, layer)
  int32_t max_batch;
  int32_t mirror_chunks;           // chunks a host mirror is laid out for: 0 = those of the placed clip, else the capacity (streaming audio)
  int32_t kv8;                     // the tidal tier (host mirror, slot pool) holds e4m3 bytes with a power-of-two scale per (chunk, head, K|V)
  long long text_seq_stride, anchor_seq_stride, pool_seq_stride, fixed_seq_stride;  // elements
  float scale_log2;                // softmax scale * log2(e)
};

struct CacheView {
  Geometry geo;
  const uint8_t *roles;      // [L][Hkv]
  const int16_t *role_idx;   // [L][Hkv] index among the heads of the same role in that layer
  const LayerInfo *layers;   // [L]
  const int32_t *upd_list;   // concatenated per-layer update lists
  const int32_t *anchor_layers;  // layers that have anchor heads, ascending
  int32_t n_anchor_layers;
  int32_t scope_global;          // tidal layers rank by the sum over all anchor layers (src = -2 in their LayerInfo)
  bf16 *text, *anchor, *pool, *fixed;
  int32_t *text_len, *T_a, *C, *S;   // [B]  (S: all slots of a tidal table)
  int32_t *S_base;                   // [B] slots filled at prefill (= S under the hard budget); what fixed heads keep
  long long *steps;                  // [B]
  long long *step_snap;              // [B][L] the step index as the layer's attention kernel saw it: what the layer's
                                     // selection kernel stamps with (the step-end update may overtake that kernel)
  int32_t *slot_chunk;               // [2][B][L][S_max]: the table a step's attention reads is copy (steps[b] & 1); the step's
                                     //   selection writes the other copy, which the step's end makes current
  int32_t *chunk_slot;               // [B][L][C_max]
  long long *stamp;                  // [B][L][S_max]
  float *score_sum;                  // [B][L][C_max]
  int32_t *sel, *n_sel;              // [B][L][topk], [B][L]
  int32_t *plan, *n_plan;            // [B][L][plan_cap][2] (chunk, slot), [B][L]
  int32_t *fixed_chunks, *fixed_n;   // [B][F_tot][FB], [B][F_tot]
  int2 *tok_m;                       // [B][L][Hkv] token-granular tidal base: kept positions of a full / the last segment;
                                     //   x < 0: they differ by segment (global top-k variant), see seg_kept
  int32_t *seg_kept;                 // [B][tidal heads over all layers][C_max] kept positions of every segment
  int32_t tid_total;                 // tidal heads over all layers
  float *pre;                        // [B][L][Hkv][C_max]
  unsigned long long *stats;         // [B][4] hits, misses, evictions, recall_bytes
  bf16 **mirror;                     // [B] pinned host mirrors (device-visible addresses)
  int8_t *kv_exp;                    // [B][tidal heads over all layers][C_max][K|V] e4m3 tidal tier: the chunk's scale exponent
  int32_t *status;
};

// ---- address helpers (element offsets; every row is d bf16) ----
__host__ __device__ inline long long text_off(const Geometry &G, int b, int l, int h, int kv) {
  return (long long)b * G.text_seq_stride + ((long long)(l * G.Hkv + h) * 2 + kv) * G.T_cap_pad * G.d;
}
__host__ __device__ inline long long anchor_off(const Geometry &G, long long seq_stride, int b, int head, int kv) {
  return (long long)b * seq_stride + ((long long)head * 2 + kv) * G.T_a_pad * G.d;
}
__host__ __device__ inline long long pool_off(const Geometry &G, const LayerInfo &li, int b, int slot, int t_idx, int kv) {
  return (long long)b * G.pool_seq_stride + li.pool_off + ((long long)(slot * li.n_tidal + t_idx) * 2 + kv) * G.ncp * G.d;
}
__host__ __device__ inline long long fixed_off(const Geometry &G, const LayerInfo &li, int b, int f_idx, int kv) {
  return (long long)b * G.fixed_seq_stride + ((long long)(li.fixed_off + f_idx) * 2 + kv) * G.FB * G.ncp * G.d;
}
// slot table of (sequence, layer) in the copy of the given parity (element offset into slot_chunk)
__host__ __device__ inline long long slot_table_off(const Geometry &G, int parity, long long bl) {
  return ((long long)parity * G.max_batch * G.L + bl) * G.S_max;
}
// compact store of a head by its index among the heads that have one (fixed heads first, then tidal token bases)
__host__ __device__ inline long long compact_off(const Geometry &G, int b, int head, int kv) {
  return (long long)b * G.fixed_seq_stride + ((long long)head * 2 + kv) * G.FB * G.ncp * G.d;
}
// C_b: the chunks the sequence's mirror is laid out for (mirror_chunks_of)
__host__ __device__ inline int mirror_chunks_of(const Geometry &G, int C_b) { return G.mirror_chunks ? G.mirror_chunks : C_b; }
__host__ __device__ inline long long mirror_off(const Geometry &G, const LayerInfo &li, int C_b, int c, int t_idx, int kv) {
  return (((long long)C_b * li.tid_prefix + (long long)c * li.n_tidal + t_idx) * 2 + kv) * G.ncp * G.d;
}

// ---- e4m3 tidal tier ----
// Offsets into the pool and the mirrors count ELEMENTS; an element is one byte there (two as bf16).
__host__ __device__ inline int tidal_elem_bytes(const Geometry &G) { return G.kv8 ? 1 : 2; }
__host__ __device__ inline long long kv_exp_off(const Geometry &G, int tid_total, int b, int tidal_head, int chunk) {
  return (((long long)b * tid_total + tidal_head) * G.C_max + chunk) * 2;
}
// Where element e (0..15) of a 16-element group of a row sits among the group's 16 bytes.  The order is chosen so that
// ldmatrix on the byte tile hands every lane exactly the elements its mma fragment wants:
//   K rows (A operand of S^T = K q^T, not transposed): lane t of a quad gets bytes 4t..4t+3 and needs elements
//     2t, 2t+1 (k-columns of its first register) and 2t+8, 2t+9 (of its third);
//   V rows (A operand of O^T = V^T P^T, transposed on the way out of shared memory in 16-bit units): the unit a lane
//     gets holds the elements j and j+8 of the d-tile (its accumulator rows).
__host__ __device__ inline int e4m3_store_pos(int kv, int e) {
  if (kv) return (e & 7) * 2 + (e >> 3);
  const int t = (e & 7) >> 1;
  return 4 * t + (e & 1) + ((e >> 3) << 1);
}

// shared-memory workspace of one table update in the selection kernel: keys[C] u64, stamp[S] i64, slot[S] i32, scores[C] f32
__host__ __device__ inline size_t select_ws_bytes(int C, int S) {
  return ((size_t)C * 8 + (size_t)S * 8 + (size_t)S * 4 + (size_t)C * 4 + 15) / 16 * 16;
}

// ---- attention launch ----
enum { ATTN_DECODE = 0, ATTN_FULL = 1, ATTN_PREFILL = 2 };

// TMA descriptors of the K/V stores, each viewed as a 2-D bf16 tensor [rows][d] with 16 x 64-element boxes and the
// 128-byte swizzle.  `anchor` is whichever store plays the contiguous full-audio role in the launch.
struct TmaMaps { CUtensorMap text, anchor, pool, fixed; };

struct AttnArgs {
  int32_t mode;          // ATTN_*
  int32_t layer;
  LayerInfo li;          // cv.layers[layer], by value (no global load on the critical path)
  int32_t n_active;
  int32_t has_new;       // k_new/v_new hold one more text row per sequence (appended by this launch)
  int32_t score_on;      // write per-granule softmax-mass partials for anchor-like heads
  const int32_t *active; // [n_active] sequence ids
  const WorkItem *items;         // device copy of the items
  const WorkItem *items_host;    // host copy (the launcher inlines short lists into the kernel parameters)
  const TmaMaps *maps;           // host pointer; passed to the kernel by value
  int32_t n_items;
  const int32_t *order;          // persistent schedule (throughput regime), else null: order[cta_ranges[c] .. cta_ranges[c+1]) are
  const int32_t *cta_ranges;     //   the item indices CTA c processes; n_ctas CTAs are launched
  int32_t n_ctas;
  int32_t throughput;            // items were cut for the 4-warp, 2-CTAs-per-SM variant (more than one wave of work)
  const int32_t *wait_epoch;     // replayed steps: tidal CTAs wait until *wait_epoch >= *expect_epoch (this layer's recall of the
  const int32_t *expect_epoch;   //   previous step, which runs outside the captured graph, has landed); null otherwise
  int32_t pdl;                   // launch with programmatic stream serialization (previous stream op is a layer kernel)
  int xpref;        // the CTAs serve several work items each and keep their copy pipeline running across them
  int wait_inputs;  // q/k_new/v_new come from the preceding work on the stream: wait for it before reading them
  const HeadItems *head_items;  // [n_active][Hkv] work items of each head (first is relative to `items`)
  const bf16 *q;         // [n_active][Hq][d]
  const bf16 *k_new, *v_new;    // [n_active][Hkv][d] or null
  // anchor-like source: decode -> cache anchor store; full -> same store, head = l*Hkv+h; prefill -> staging, head = h
  const bf16 *anchor_base;
  long long anchor_seq_stride;
  int32_t anchor_head0;
  // split partials
  float *part_o;         // [n_items][g][d]
  float2 *part_ml;       // [n_items][g]   (m in log2 units, l)
  float2 *gran_em;       // [n_active][n_aq][n_ag_max]  (sum of 2^(s-m) over the granule, m at that time)
  int32_t n_aq, n_ag_max;
  // fused head merge (decode and full modes)
  int32_t *head_done;    // [n_active][Hkv] finished-item counters (self-resetting)
  float2 *head_mz;       // [n_active][Hq] final (M, Z) per query head
  bf16 *out;             // [n_active][Hq][d]
};

// Several layers in one launch: per-layer arguments and the first CTA of each layer's range.
constexpr int MULTI_LAYERS_MAX = 48;
struct MultiArgs {
  int32_t n;
  int32_t cta_prefix[MULTI_LAYERS_MAX + 1];
  int32_t cta_first[MULTI_LAYERS_MAX];   // the layer's first CTA in this launch (a launch may carry a part of its CTAs)
  AttnArgs l[MULTI_LAYERS_MAX];
};

// Selection launch (side stream): chunk scores of `layer` from its granule partials, then top-k, residency update
// and recall plan for every layer in the update list.  Static data travels by value.
struct SelectArgs {
  int32_t layer, n_active, score_on;
  int32_t do_score, do_update;   // which half of the work this launch does (both, unless the step splits them)
  LayerInfo li;
  const int32_t *active;
  const float2 *gran_em;   // this layer's [n_active][n_aq][n_ag_max]
  const float2 *head_mz;   // this layer's [n_active][Hq]
  int32_t n_aq, n_ag_max;
  uint8_t aq_head[MAX_AQ]; // query-head index of anchor q-head slot aq (score order)
  int16_t upd_layer[MAX_UPD_BY_VALUE], upd_src[MAX_UPD_BY_VALUE];
  // Captured steps: the selection CTA that finishes last in the step also does the step's bookkeeping (step counters,
  // text lengths, recall epoch), which saves the dependent launch of a kernel of its own at the end of every step.
  int32_t fold_total;      // selection CTAs in the step (0: the step-end kernel runs instead)
  int32_t fold_appended;   // the step appended a text token
  int32_t *fold_counter;   // finished selection CTAs (self-resetting)
  int32_t *fold_bump_epoch;
  // Recall outside the captured step: a layer whose tables need no copy in this step (for any sequence) gets its recall
  // epoch published right here, so the next step's tidal CTAs do not wait for the recall launch at all.
  int32_t *epoch_words;        // [L] or null
  int32_t *empty_ctr;          // [L] sequences with an empty plan (reset by whoever publishes the layer's epoch)
  const int32_t *step_epoch;
  // Selection that runs beside the step's tidal attention (all layers issued together): the step count is read live (the
  // snapshot of a layer whose first head is tidal may not be written yet) and, before a layer's plan is rewritten, the
  // recall of the previous step must be done with it (bounded wait on the layer's epoch word).
  int32_t overlapped;
};

// Completion signalling of a recall launch that runs outside the captured step (all null for in-step launches).
struct RecallSignal {
  int32_t *epoch_words;       // [L] epoch of the last completed recall of each layer's table
  int32_t *counters;          // [L] finished-CTA counters (self-resetting)
  int32_t *empty_ctr;         // [L] the selection kernels' empty-plan counters, reset here
  int32_t publish_epoch;      // epoch to publish: the number of replayed steps that have ended with this one (the host counts
                              // them; the device word may already be further when this kernel runs late)
};

// kernels' host launchers (defined in the .cu files)
cudaError_t launch_attn(const CacheView &cv, const AttnArgs &a, cudaStream_t st);
// groups: CTAs per sequence (a layer that updates many tables, e.g. the last one under the global score scope)
cudaError_t launch_select(const CacheView &cv, const SelectArgs &a, size_t smem_bytes, int groups, cudaStream_t st);
cudaError_t launch_select_all(const CacheView &cv, const SelectArgs *layer_args_dev, const int4 *map_dev, int n_entries,
                              const SelectArgs &step, size_t smem_bytes, cudaStream_t st);
// the same with the layers' arguments and the map in the kernel parameters (no global load before the CTA knows its
// work); n_layers <= SELECT_TABLE_LAYERS and n_entries <= SELECT_TABLE_ENTRIES
constexpr int SELECT_TABLE_LAYERS = 48, SELECT_TABLE_ENTRIES = 64;
struct SelectAllTable { int4 map[SELECT_TABLE_ENTRIES]; SelectArgs l[SELECT_TABLE_LAYERS]; };
cudaError_t launch_select_all_params(const CacheView &cv, const SelectArgs *layer_args_host, int n_layers, const int4 *map_host,
                                     int n_entries, const SelectArgs &step, size_t smem_bytes, cudaStream_t st);
cudaError_t launch_step_end(const CacheView &cv, int n_active, const int32_t *active, int appended, int32_t *bump_epoch,
                            cudaStream_t st);
cudaError_t launch_recall(const CacheView &cv, int n_active, const int32_t *active, const int32_t *layers_dev, int n_layers,
                          int skip_copy, RecallSignal sig, cudaStream_t st);
cudaError_t launch_place_scatter(const CacheView &cv, int b, int layer, const bf16 *k, const bf16 *v, int n_tokens, int ab,
                                 int ae, int T_t, int C_b, int S_b, int S_base, bf16 *stage, cudaStream_t st);
cudaError_t launch_prefill_select(const CacheView &cv, int b, int layer, const HeadItems *head_items, const float2 *part_ml,
                                  const float2 *gran_em, int n_ag_max, int first, int last, cudaStream_t st);
cudaError_t launch_place_gather(const CacheView &cv, int b, int layer, int full_mode, const bf16 *stage, int C_b,
                                cudaStream_t st);
// token-granular compression of the layer's fixed heads (after the chunk-granular placement staged the prefix)
cudaError_t launch_token_compress(const CacheView &cv, int b, int layer, int n_comp, int n_tidal_base, const bf16 *stage,
                                  const bf16 *q_text, int n_q, int T_t, int T_a, int seg, const float *retention_dev,
                                  int variant, float *work, float *p_tok, int32_t *flags, long long p_stride,
                                  int32_t *fixed_tok, int tok_cap, int32_t *tok_n, cudaStream_t st);
cudaError_t launch_append_audio(const CacheView &cv, int b, int layer, int full_mode, const bf16 *k, const bf16 *v, int n_tokens,
                                int T_a_old, int S_old, int set_dims, int T_a_new, int C_new, int S_new, cudaStream_t st);
cudaError_t launch_exchange_scores(const CacheView &cv, int n_active, const int32_t *active, float *buf, int out, cudaStream_t st);
cudaError_t launch_prefill_tidal_sum(const CacheView &cv, int b, int layer, float *dst, cudaStream_t st);
cudaError_t launch_prefill_retable(const CacheView &cv, int b, int layer, const float *sums, cudaStream_t st);
cudaError_t launch_copy_plan(const uint4 *src_host_mapped, uint4 *dst, long long n_vec, int n_ctas, cudaStream_t st);
cudaError_t configure_attn_kernels();
// the CTAs of several layers' launches (one-shot variant) in one launch
// CTAs [first[l], first[l] + count[l]) of every layer l (null: all of them); pdl: launched programmatically dependent on
// what precedes it in the stream
cudaError_t launch_attn_multi(const CacheView &cv, const AttnArgs *args, int n, const int *first, const int *count, bool pdl,
                              cudaStream_t st);
// Encodes the descriptor of one store: base (device), rows, head_dim.  Returns false if the driver refuses.
bool encode_store_map(CUtensorMap *map, const void *base, unsigned long long rows, int d);
// the slot pool as e4m3: rows of 128 bytes, boxes of 16 rows, 128-byte swizzle
bool encode_store_map_e4m3(CUtensorMap *map, const void *base, unsigned long long rows);
// e4m3 tidal tier, at placement: per (chunk, tidal head, K|V) the scale exponent from the staged rows, which are then
// replaced by the values their bytes decode to
cudaError_t launch_quantise_stage(const CacheView &cv, int b, int layer, bf16 *stage, int C_b, cudaStream_t st);
cudaError_t configure_select_kernel();
constexpr int SELECT_SMEM_CAP = 200 * 1024;  // dynamic shared memory the selection kernel may be launched with
bool attn_xpref_fits(int g, int d);  // a one-shot CTA can hold its merge scratch behind the copy stages
int attn_warps(bool throughput);  // warps per attention CTA in the latency / throughput variant
int attn_persistent_ctas_per_sm(int g, int d);  // persistent (throughput-variant) CTAs that fit one SM

}  // namespace wnw
