// Host runtime behind the C ABI of include/wnw.h: cache object, device stores, work lists, streams and events.
// Every step of the path runs in the kernels of wnw_attn.cu / wnw_kernels.cu; this file only validates
// arguments, sizes buffers and queues launches.  There is no CPU fallback.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/wnw.h"
#include "../../include/wnw_debug.h"
#include "wnw_internal.cuh"

using namespace wnw;

namespace {

struct SeqHost {
  int placed_layers = 0;
  int T_a = 0, T_t = 0, C = 0, S = 0, S_base = 0;   // S: all slots of a tidal table; S_base: the permanent ones
  int T_a_fixed = 0, S_fixed = 0;   // the clip and the slot count at placement: what a fixed head keeps for good (streaming audio)
  int append_layer = 0, append_n = 0;   // an append of audio in progress: layers done, positions per layer
  bf16 *mirror = nullptr;
  size_t mirror_bytes = 0;
  std::vector<int> fixed_blocks;   // [L][Hkv] blocks of a token-compacted head's store; empty or -1: S_base chunks
  std::vector<int2> tok_m;         // [L][Hkv] tidal token bases: kept positions of a full / of the last segment
};

struct LayerWork {
  int first_item = 0, n_items = 0, max_count = 0;  // range in the uploaded item array
  bool throughput = false;                         // which kernel variant the items were cut for
  size_t part_off = 0;                             // first partial of this layer in the partial buffers (in items)
  int n_ctas = 0, order_off = 0, ranges_off = 0;   // items per CTA (persistent schedule, or packed short heads): offsets
  int n_ctas_free = 0;   // BATCHED layers: the first n_ctas_free CTAs hold no tidal head (they need no recall epoch) ...
  int n_ctas_anchor = 0; // ... and the first n_ctas_anchor of those hold the anchor heads (what the step's selection waits for)
  bool packed = false;                             // one-shot CTAs that serve several short heads each
  int head_items_off = 0;                          // offset in the uploaded HeadItems array
};

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

}  // namespace

struct wnw_cache {
  wnw_config_t cfg;
  Geometry geo;
  CacheView cv;
  std::vector<uint8_t> roles;
  std::vector<int16_t> role_idx;
  std::vector<LayerInfo> layers;
  std::vector<int32_t> upd_list, anchor_layers;
  std::vector<int> tail_of;  // layer -> layer whose tail updates its table, -1 if none
  std::vector<uint8_t> anchor_layer;   // [L] the layer has an anchor head (on any shard, when the cache holds one shard of the heads)
  bool scores_exported = false, scores_imported = false;   // head-sharded step: where the exchange stands
  int tid_total = 0, n_sm = 148;
  std::vector<SeqHost> seqs;
  std::vector<void *> dev_allocs;
  std::vector<bf16 *> mirror_ptrs;  // host copy of cv.mirror
  bf16 *stage = nullptr;
  TmaMaps maps_decode, maps_prefill;  // TMA descriptors: cache stores; prefill scoring reads the staging copy as `anchor`
  int32_t *d_iota = nullptr, *d_active = nullptr;
  // step state
  std::vector<int> active;
  bool in_step = false;
  int next_layer = 0, appended = -1;
  // work lists
  std::vector<int> wl_active;
  std::vector<int> wl_T_a;
  std::vector<LayerWork> wl_layers;
  WorkItem *d_items = nullptr;
  int32_t *d_sched = nullptr, *d_pf_sched = nullptr;  // persistent schedules: [order of all layers | ranges of all layers]
  size_t d_sched_cap = 0, sched_ranges_base = 0, pf_sched_cap = 0, pf_ranges_base = 0;
  int pf_n_ctas = 0;
  std::vector<WorkItem> h_items, h_pf_items;  // host copies (short lists are inlined into kernel parameters)
  HeadItems *d_head_items = nullptr;
  size_t d_items_cap = 0, d_head_items_cap = 0;
  int prefill_seq = -1, prefill_T_a = -1;
  WorkItem *d_pf_items = nullptr;
  HeadItems *d_pf_head_items = nullptr;
  int pf_n_items = 0;
  bool pf_throughput = false;
  size_t pf_items_cap = 0;
  // partial buffers
  float *part_o = nullptr;
  float2 *part_ml = nullptr, *gran_em = nullptr, *head_mz = nullptr;
  int32_t *head_done = nullptr;
  float2 *pf_gran_em = nullptr, *pf_part_ml = nullptr;
  float *pf_part_o = nullptr;
  size_t part_cap_total = 0;
  int part_cap_items = 0, n_aq_max = 0, n_ag_max = 0;
  // streams / events
  static constexpr int N_SIDE = 8;  // layers alternate between side streams so selection + recall keep pace with attention
  cudaStream_t side[N_SIDE] = {}, last_stream = nullptr;
  std::vector<cudaEvent_t> ev_layer_done, ev_side_done;
  std::vector<cudaEvent_t> ev_layer_done_cap, ev_side_done_cap;  // used only inside a stream capture
  std::vector<char> side_recorded;
  std::vector<size_t> sel_smem;   // dynamic shared memory of each layer's selection launch
  size_t gran_em_layer_stride = 0;
  bool step_capturing = false;
  // Captured steps of small launches: the selection work of all layers in one launch at the end of the step (two when a
  // layer ranks by another layer's scores: first all scores, then all updates).
  bool cap_select_all = false, select_single_ok = false;
  SelectArgs *d_sel_args = nullptr;
  int4 *d_sel_map = nullptr;
  std::vector<SelectArgs> h_sel_args;   // host copies: small stacks pass them in the kernel parameters
  std::vector<int4> h_sel_map;
  int sel_map_single[2] = {0, 0}, sel_map_score[2] = {0, 0}, sel_map_update[2] = {0, 0};   // offset, entries
  size_t sel_all_smem = 0;
  bool cap_fold = false;   // captured steps: the last selection CTA closes the step
  int n_side_layers = 0, n_select_ctas = 0;   // layers with a selection kernel; its CTAs per sequence over all layers
  int32_t *d_fold_ctr = nullptr, *d_empty_ctr = nullptr;
  int32_t host_epoch = 0;   // replayed steps with out-of-graph recall so far = the value of the device's step epoch after them
  long long launches[4] = {0, 0, 0, 0}, cap_launches[4] = {0, 0, 0, 0};  // attention, selection, recall, step-end kernels
  void count_launch(int kind, int n, bool capturing) { (capturing ? cap_launches : launches)[kind] += n; }
  int layer_dependency = WNW_LAYERS_INDEPENDENT;
  std::vector<AttnArgs> batch_args;   // BATCHED layers of a captured step: recorded per layer, launched by the last one
  bool cap_batched = false;
  // the step's selection beside its tidal attention (all layers issued together, two parts): forked after the first part
  bool cap_sel_overlap = false;
  cudaEvent_t ev_sel_fork = nullptr, ev_sel_join = nullptr;
  int batched_target = 0;             // granules of work per CTA when the step's layers share one launch ...
  int batched_target_tidal = 0;       // ... and per CTA of its second part, the tidal heads
  // replayed steps: one recall launch per step outside the captured graph, overlapping the next step
  int32_t *d_recall_epoch = nullptr, *d_recall_ctr = nullptr, *d_step_epoch = nullptr;
  bool cap_external_recall = false, graph_external_recall = false, recall_all_pending = false;
  cudaEvent_t ev_graph_done = nullptr, ev_recall_all = nullptr;
  static constexpr int direct_max_granules = 64;   // scale of the one-CTA rule: a head of up to 2x (overlapping layers) or x/2
                                                   // (chained layers) this many granules (text capacity included) is not split
  // captured step
  bool graph_capturing = false;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t graph_exec = nullptr;
  std::vector<int> graph_active, graph_prepared;
  long long wl_epoch = 0, graph_epoch = -1;  // work-list generation the graph was captured against
  int graph_appended = 0;
  int last_side_layer[N_SIDE] = {-1, -1, -1, -1, -1, -1, -1, -1};

  cudaEvent_t ev_place = nullptr, ev_step = nullptr;
  bool place_recorded = false, step_recorded = false;
  // token-granular compression of fixed heads (allocated by the first wnw_place_prefill_tokens)
  float *tok_work = nullptr, *tok_p = nullptr, *tok_ret = nullptr;
  int32_t *tok_flags = nullptr, *fixed_tok = nullptr, *tok_n = nullptr;
  int tok_cap = 0, tok_fixed_max = 0, tok_last_seq = -1, tok_last_layer = -1;
  long long tok_p_stride = 0;
  // timing
  bool timing = false;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> t_used;
  std::vector<cudaEvent_t> t_free;
  cudaError_t last_cuda = cudaSuccess;
};

#define CK(expr)                                 \
  do {                                           \
    cudaError_t _e = (expr);                     \
    if (_e != cudaSuccess) {                     \
      c->last_cuda = _e;                         \
      return _e == cudaErrorMemoryAllocation ? WNW_ERR_OOM_DEVICE : WNW_ERR_CUDA; \
    }                                            \
  } while (0)

// CTAs per sequence of a layer's selection kernel: one per eight tables to update.
static int select_groups(const LayerInfo &li) { return std::max(1, std::min(8, (li.upd_count + 7) / 8)); }

static int slots_for(float budget, int C) {
  if (C <= 0) return 0;
  int S = (int)std::floor((double)budget * (double)C + 1e-6);
  if (S < 1) S = 1;
  if (S > C) S = C;
  return S;
}
// All slots of a tidal table: under SEGMENT_LAG the permanent ones plus room for everything selected within the last
// evict_lag + 1 steps (two segments per chunk), so a miss always finds a free slot.  With a token-granular base no
// slot is permanent.
static bool lag_residency(const wnw_config_t &cfg) { return cfg.residency != WNW_RESIDENCY_HARD_BUDGET; }
static int base_slots_for(const wnw_config_t &cfg, int C) {
  return cfg.residency == WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE ? 0 : slots_for(cfg.budget, C);
}
static int slots_total(const wnw_config_t &cfg, int C) {
  const int base = base_slots_for(cfg, C);
  if (!lag_residency(cfg) || C <= 0) return base;
  return base + std::min(2 * cfg.topk * (cfg.evict_lag + 1), C - base);
}
// Blocks of chunk_tokens rows in a head's compact store (fixed heads; tidal token bases): the budget's share plus, under
// the lag residencies, as many blocks again as a table has dynamic slots (per-head retentions spread around the budget).
static int compact_blocks(const wnw_config_t &cfg, int C) {
  const int base = slots_for(cfg.budget, C);
  if (!lag_residency(cfg) || C <= 0) return base;
  return base + std::min(2 * cfg.topk * (cfg.evict_lag + 1), C - base);
}

template <typename T>
static wnw_status_t dev_alloc(wnw_cache *c, T **p, size_t count, bool zero = true) {
  const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
  CK(cudaMalloc((void **)p, bytes));
  c->dev_allocs.push_back((void *)*p);
  if (zero) CK(cudaMemset(*p, 0, bytes));
  return WNW_OK;
}
template <typename T>
static wnw_status_t dev_upload(wnw_cache *c, T **p, const std::vector<T> &v) {
  wnw_status_t s = dev_alloc(c, p, v.size(), true);
  if (s != WNW_OK) return s;
  if (!v.empty()) CK(cudaMemcpy(*p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice));
  return WNW_OK;
}

static void destroy_impl(wnw_cache *c) {
  DeviceGuard guard(c->cfg.device);
  cudaDeviceSynchronize();
  for (void *p : c->dev_allocs) cudaFree(p);
  for (auto &s : c->seqs)
    if (s.mirror) cudaFreeHost(s.mirror);
  for (auto sd : c->side)
    if (sd) cudaStreamDestroy(sd);

  for (auto e : c->ev_layer_done) cudaEventDestroy(e);
  for (auto e : c->ev_side_done) cudaEventDestroy(e);
  for (auto e : c->ev_layer_done_cap) cudaEventDestroy(e);
  for (auto e : c->ev_side_done_cap) cudaEventDestroy(e);
  if (c->ev_sel_fork) cudaEventDestroy(c->ev_sel_fork);
  if (c->ev_sel_join) cudaEventDestroy(c->ev_sel_join);
  if (c->ev_place) cudaEventDestroy(c->ev_place);
  if (c->ev_step) cudaEventDestroy(c->ev_step);
  if (c->ev_graph_done) cudaEventDestroy(c->ev_graph_done);
  if (c->ev_recall_all) cudaEventDestroy(c->ev_recall_all);
  if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
  if (c->graph) cudaGraphDestroy(c->graph);
  for (auto &p : c->t_used) { cudaEventDestroy(p.first); cudaEventDestroy(p.second); }
  for (auto e : c->t_free) cudaEventDestroy(e);
  delete c;
}

extern "C" const char *wnw_status_string(wnw_status_t s) {
  switch (s) {
    case WNW_OK: return "ok";
    case WNW_ERR_INVALID_ARG: return "invalid argument";
    case WNW_ERR_STATE: return "call out of order for the cache's state";
    case WNW_ERR_OOM_DEVICE: return "out of device memory";
    case WNW_ERR_OOM_HOST: return "out of pinned host memory";
    case WNW_ERR_CUDA: return "CUDA runtime error";
    case WNW_ERR_CAPACITY: return "sequence capacity exceeded";
    case WNW_ERR_TIMEOUT: return "timeout";
    case WNW_ERR_UNSUPPORTED: return "unsupported shape";
    case WNW_ERR_DEVICE_CHECK: return "device-side consistency check failed";
  }
  return "unknown status";
}

static wnw_status_t validate_config(const wnw_config_t *cfg) {
  if (!cfg || !cfg->roles) return WNW_ERR_INVALID_ARG;
  if (cfg->n_layers < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads) return WNW_ERR_INVALID_ARG;
  if (cfg->max_batch < 1 || cfg->max_audio_tokens < 0 || cfg->max_text_tokens < 0) return WNW_ERR_INVALID_ARG;
  if (cfg->max_audio_tokens + cfg->max_text_tokens < 1) return WNW_ERR_INVALID_ARG;
  if (cfg->chunk_tokens < 1 || cfg->topk < 0 || cfg->topk > MAX_TOPK || cfg->evict_lag < 0) return WNW_ERR_INVALID_ARG;
  if (!(cfg->budget > 0.f && cfg->budget <= 1.f)) return WNW_ERR_INVALID_ARG;
  if (!(cfg->softmax_scale >= 0.f) || std::isinf(cfg->softmax_scale)) return WNW_ERR_INVALID_ARG;
  if (cfg->mode != WNW_MODE_TIERED && cfg->mode != WNW_MODE_FULL) return WNW_ERR_INVALID_ARG;
  if (cfg->score_scope != WNW_SCOPE_PER_LAYER && cfg->score_scope != WNW_SCOPE_GLOBAL) return WNW_ERR_INVALID_ARG;
  if (cfg->residency < WNW_RESIDENCY_HARD_BUDGET || cfg->residency > WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE) return WNW_ERR_INVALID_ARG;
  if (cfg->recall_mode < WNW_RECALL_SIDE_STREAM || cfg->recall_mode > WNW_RECALL_SKIP) return WNW_ERR_INVALID_ARG;
  if (cfg->device < 0 || cfg->streaming_audio < 0 || cfg->streaming_audio > 1) return WNW_ERR_INVALID_ARG;
  if (cfg->defer_selection < 0 || cfg->defer_selection > 1) return WNW_ERR_INVALID_ARG;
  if (cfg->defer_selection && (cfg->score_scope != WNW_SCOPE_PER_LAYER || cfg->residency != WNW_RESIDENCY_HARD_BUDGET ||
                               cfg->recall_mode == WNW_RECALL_INLINE))
    return WNW_ERR_UNSUPPORTED;
  bool any_anchor = false, any_tidal = false;
  for (int i = 0; i < cfg->n_layers * cfg->n_kv_heads; ++i) {
    if (cfg->roles[i] > WNW_ROLE_FIXED) return WNW_ERR_INVALID_ARG;
    any_anchor |= cfg->roles[i] == WNW_ROLE_ANCHOR;
    any_tidal |= cfg->roles[i] == WNW_ROLE_TIDAL;
    // a layer the model-wide flags call anchor-less cannot hold an anchor head here
    if (cfg->global_anchor_layers && cfg->roles[i] == WNW_ROLE_ANCHOR && !cfg->global_anchor_layers[i / cfg->n_kv_heads]) return WNW_ERR_INVALID_ARG;
  }
  if (cfg->global_anchor_layers)
    for (int l = 0; l < cfg->n_layers; ++l) any_anchor |= cfg->global_anchor_layers[l] != 0;
  if (cfg->mode == WNW_MODE_TIERED && any_tidal && !any_anchor) return WNW_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return WNW_ERR_UNSUPPORTED;
  if (cfg->tidal_kv_format != WNW_TIDAL_KV_BF16 && cfg->tidal_kv_format != WNW_TIDAL_KV_FP8_E4M3) return WNW_ERR_INVALID_ARG;
  // e4m3 tidal tier: one swizzle atom per row (head_dim 128); a chunk's scale is fixed when the chunk is placed
  if (cfg->mode == WNW_MODE_TIERED && cfg->tidal_kv_format == WNW_TIDAL_KV_FP8_E4M3 &&
      (cfg->head_dim != 128 || cfg->residency == WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE || cfg->streaming_audio))
    return WNW_ERR_UNSUPPORTED;
  if (cfg->n_q_heads / cfg->n_kv_heads > MAX_G || cfg->n_q_heads > MAX_AQ || cfg->n_layers > 32767) return WNW_ERR_UNSUPPORTED;
  return WNW_OK;
}

static SelectArgs static_select_args(const wnw_cache *c, int layer);

extern "C" wnw_status_t wnw_create(const wnw_config_t *cfg, wnw_cache_t **out) {
  if (!out) return WNW_ERR_INVALID_ARG;
  wnw_status_t vs = validate_config(cfg);
  if (vs != WNW_OK) return vs;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device >= n_dev) return WNW_ERR_CUDA;
  wnw_cache *c = new (std::nothrow) wnw_cache();
  if (!c) return WNW_ERR_OOM_HOST;
  c->cfg = *cfg;
  if (c->cfg.topk == 0) c->cfg.topk = 3;
  DeviceGuard guard(cfg->device);
  auto fail = [&](wnw_status_t s) { destroy_impl(c); return s; };
#define CKC(call) do { wnw_status_t _s = (call); if (_s != WNW_OK) return fail(_s); } while (0)
#define CKE(expr) do { cudaError_t _e = (expr); if (_e != cudaSuccess) { return fail(_e == cudaErrorMemoryAllocation ? WNW_ERR_OOM_DEVICE : WNW_ERR_CUDA); } } while (0)
  cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, cfg->device);
  CKE(configure_attn_kernels());
  CKE(configure_select_kernel());
  const int L = cfg->n_layers, Hkv = cfg->n_kv_heads, d = cfg->head_dim, nc = cfg->chunk_tokens;
  const bool full = cfg->mode == WNW_MODE_FULL;
  c->roles.assign(cfg->roles, cfg->roles + (size_t)L * Hkv);
  c->cfg.roles = nullptr;
  c->anchor_layer.assign(L, 0);
  for (int l = 0; l < L; ++l) {
    bool has = cfg->global_anchor_layers ? cfg->global_anchor_layers[l] != 0 : false;
    for (int h = 0; h < Hkv && !cfg->global_anchor_layers; ++h) has = has || cfg->roles[l * Hkv + h] == WNW_ROLE_ANCHOR;
    c->anchor_layer[l] = has;
  }
  c->cfg.global_anchor_layers = nullptr;
  Geometry &G = c->geo;
  G.L = L; G.Hq = cfg->n_q_heads; G.Hkv = Hkv; G.d = d; G.g = cfg->n_q_heads / Hkv; G.nc = nc; G.ncp = (nc + GR - 1) / GR * GR; G.gpc = G.ncp / GR;
  G.topk = c->cfg.topk;
  G.T_cap_pad = (std::max(cfg->max_text_tokens, 1) + GR - 1) / GR * GR;
  G.n_tg = G.T_cap_pad / GR;
  G.C_max = (cfg->max_audio_tokens + nc - 1) / nc;
  G.S_max = full ? 0 : slots_total(c->cfg, G.C_max);
  G.FB = full ? 0 : compact_blocks(c->cfg, G.C_max);
  G.lag_mode = !full && lag_residency(c->cfg);
  G.token_base = !full && c->cfg.residency == WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE;
  G.delta = c->cfg.evict_lag;
  G.plan_cap = G.lag_mode ? 2 * G.topk : G.topk;
  G.T_a_pad = std::max(G.C_max, 1) * G.ncp;
  G.max_batch = cfg->max_batch;
  G.mirror_chunks = (!full && cfg->streaming_audio) ? G.C_max : 0;
  G.kv8 = !full && cfg->tidal_kv_format == WNW_TIDAL_KV_FP8_E4M3;
  const double scale = cfg->softmax_scale > 0.f ? (double)cfg->softmax_scale : 1.0 / std::sqrt((double)d);
  G.scale_log2 = (float)(scale * 1.4426950408889634);
  // roles -> per-layer tables, score routing, update lists
  c->role_idx.assign((size_t)L * Hkv, 0);
  c->layers.assign(L, LayerInfo{});
  int a_tot = 0, f_tot = 0, t_tot = 0;
  long long pool_elems = 0;
  for (int l = 0; l < L; ++l) {
    LayerInfo &li = c->layers[l];
    li.anchor_off = a_tot; li.fixed_off = f_tot; li.tid_prefix = t_tot; li.pool_off = pool_elems; li.src = -1;
    for (int h = 0; h < Hkv; ++h) {
      const int role = c->roles[l * Hkv + h];
      int16_t &ri = c->role_idx[l * Hkv + h];
      if (role == ROLE_ANCHOR) ri = (int16_t)li.n_anchor++;
      else if (role == ROLE_TIDAL) ri = (int16_t)li.n_tidal++;
      else ri = (int16_t)li.n_fixed++;
    }
    a_tot += li.n_anchor; f_tot += li.n_fixed; t_tot += li.n_tidal;
    pool_elems += (long long)G.S_max * li.n_tidal * 2 * G.ncp * d;
  }
  c->tid_total = t_tot;
  c->tail_of.assign(L, -1);
  std::vector<std::vector<int>> upd(L);
  for (int l = 0; l < L; ++l) {
    if (full || c->layers[l].n_tidal == 0) continue;
    int best = -1;
    for (int a = 0; a < L; ++a)
      if (c->anchor_layer[a] && (best < 0 || std::abs(a - l) < std::abs(best - l))) best = a;
    const bool global = cfg->score_scope == WNW_SCOPE_GLOBAL;
    c->layers[l].src = (global && best >= 0) ? -2 : best;  // nearest anchor layer, ties to the lower one; -2: the global accumulator
    const int x = global ? L - 1 : std::max(l, best);  // first point at which layer l's attention and its scores are done
    c->tail_of[l] = x;
    upd[x].push_back(l);
  }
  for (int l = 0; l < L; ++l) {
    c->layers[l].upd_first = (int)c->upd_list.size();
    c->layers[l].upd_count = (int)upd[l].size();
    c->upd_list.insert(c->upd_list.end(), upd[l].begin(), upd[l].end());
  }
  G.A_tot = full ? L * Hkv : a_tot;
  G.F_fix = full ? 0 : f_tot;
  G.F_tot = full ? 0 : f_tot + (G.token_base ? t_tot : 0);   // tidal heads keep their token base in a compact store too
  G.text_seq_stride = (long long)L * Hkv * 2 * G.T_cap_pad * d;
  G.anchor_seq_stride = (long long)G.A_tot * 2 * G.T_a_pad * d;
  G.pool_seq_stride = full ? 0 : pool_elems;
  G.fixed_seq_stride = (long long)G.F_tot * 2 * G.FB * G.ncp * d;

  CacheView &cv = c->cv;
  memset(&cv, 0, sizeof(cv));
  cv.geo = G;
  const size_t B = (size_t)cfg->max_batch;
  {
    uint8_t *p; int16_t *q; LayerInfo *li; int32_t *ul;
    CKC(dev_upload(c, &p, c->roles)); cv.roles = p;
    CKC(dev_upload(c, &q, c->role_idx)); cv.role_idx = q;
    CKC(dev_upload(c, &li, c->layers)); cv.layers = li;
    CKC(dev_upload(c, &ul, c->upd_list)); cv.upd_list = ul;
    for (int l = 0; l < L; ++l)
      if (c->layers[l].n_anchor > 0) c->anchor_layers.push_back(l);
    int32_t *al;
    CKC(dev_upload(c, &al, c->anchor_layers)); cv.anchor_layers = al;
    cv.n_anchor_layers = (int32_t)c->anchor_layers.size();
    cv.scope_global = !full && cfg->score_scope == WNW_SCOPE_GLOBAL;
  }
  CKC(dev_alloc(c, &cv.text, B * (size_t)G.text_seq_stride));
  CKC(dev_alloc(c, &cv.anchor, B * (size_t)G.anchor_seq_stride));
  CKC(dev_alloc(c, &cv.pool, G.kv8 ? (B * (size_t)G.pool_seq_stride + 1) / 2 : B * (size_t)G.pool_seq_stride));   // one byte per element as e4m3
  CKC(dev_alloc(c, &cv.kv_exp, G.kv8 ? B * (size_t)std::max(t_tot, 1) * std::max(G.C_max, 1) * 2 : 1));
  CKC(dev_alloc(c, &cv.fixed, B * (size_t)G.fixed_seq_stride));
  CKC(dev_alloc(c, &c->stage, (size_t)Hkv * 2 * G.T_a_pad * d));
  CKC(dev_alloc(c, &cv.text_len, B)); CKC(dev_alloc(c, &cv.T_a, B)); CKC(dev_alloc(c, &cv.C, B)); CKC(dev_alloc(c, &cv.S, B));
  CKC(dev_alloc(c, &cv.S_base, B));
  CKC(dev_alloc(c, &cv.steps, B));
  CKC(dev_alloc(c, &cv.step_snap, B * L));
  CKC(dev_alloc(c, &cv.slot_chunk, 2 * B * L * std::max(G.S_max, 1)));   // two copies, see slot_table_off
  CKC(dev_alloc(c, &cv.chunk_slot, B * L * std::max(G.C_max, 1)));
  CKC(dev_alloc(c, &cv.stamp, B * L * std::max(G.S_max, 1)));
  CKC(dev_alloc(c, &cv.score_sum, B * L * std::max(G.C_max, 1)));
  CKC(dev_alloc(c, &cv.sel, B * L * G.topk)); CKC(dev_alloc(c, &cv.n_sel, B * L));
  CKC(dev_alloc(c, &cv.plan, B * L * G.plan_cap * 2)); CKC(dev_alloc(c, &cv.n_plan, B * L));
  CKC(dev_alloc(c, &cv.fixed_chunks, B * std::max(G.F_tot, 1) * std::max(G.FB, 1)));
  CKC(dev_alloc(c, &cv.fixed_n, B * std::max(G.F_tot, 1)));
  CKC(dev_alloc(c, &cv.tok_m, G.token_base ? B * (size_t)L * Hkv : 1));
  CKC(dev_alloc(c, &cv.seg_kept, G.token_base ? B * (size_t)std::max(t_tot, 1) * std::max(G.C_max, 1) : 1));
  cv.tid_total = t_tot;
  CKC(dev_alloc(c, &cv.pre, B * L * Hkv * std::max(G.C_max, 1)));
  CKC(dev_alloc(c, &cv.stats, B * 4));
  CKC(dev_alloc(c, &cv.mirror, B));
  CKC(dev_alloc(c, &cv.status, 1));
  {
    std::vector<int32_t> iota(B);
    for (size_t i = 0; i < B; ++i) iota[i] = (int32_t)i;
    CKC(dev_upload(c, &c->d_iota, iota));
  }
  CKC(dev_alloc(c, &c->d_active, B));
  // partial buffers: the work-list builder keeps items <= target + heads
  int n_aq = 0;
  for (int l = 0; l < L; ++l) n_aq = std::max(n_aq, c->layers[l].n_anchor * G.g);
  c->n_aq_max = std::max(n_aq, 1);
  c->n_ag_max = std::max(G.C_max * G.gpc, 1);
  c->part_cap_items = 10 * c->n_sm + 2 * (int)B * Hkv + 64;
  // split partials of the prefill scoring pass; the decode layers get one region each (sized with the work lists),
  // because consecutive layer kernels overlap
  CKC(dev_alloc(c, &c->pf_part_o, (size_t)c->part_cap_items * G.g * d, false));
  CKC(dev_alloc(c, &c->pf_part_ml, (size_t)c->part_cap_items * G.g, false));
  // granule partials and final (M,Z) are per layer: the side-stream selection of layer l reads them while the
  // caller's stream already runs later layers
  c->gran_em_layer_stride = B * (size_t)c->n_aq_max * c->n_ag_max;
  CKC(dev_alloc(c, &c->gran_em, full ? 1 : (size_t)L * c->gran_em_layer_stride, false));
  CKC(dev_alloc(c, &c->pf_gran_em, full ? 1 : (size_t)G.Hq * c->n_ag_max, false));
  CKC(dev_alloc(c, &c->head_mz, (size_t)L * B * G.Hq, false));
  c->sel_smem.assign(L, 0);
  for (int l = 0; l < L && !full; ++l) {
    const LayerInfo &li = c->layers[l];
    const size_t n_aq_l = (size_t)std::max(li.n_anchor * G.g, 1);
    const size_t fixed_part = (n_aq_l * 8 + 15) / 16 * 16 + 2 * (((size_t)G.C_max * 4 + 15) / 16 * 16) + 16 +
                              (size_t)std::min(li.upd_count, 8) * select_ws_bytes(G.C_max, G.S_max);
    const size_t per_chunk = li.n_anchor > 0 ? n_aq_l * G.gpc * 8 : 0;
    const size_t cap = SELECT_SMEM_CAP - 16;
    if (fixed_part + per_chunk > cap) return fail(WNW_ERR_UNSUPPORTED);  // chunk tables too large for one CTA
    c->sel_smem[l] = std::min(cap, fixed_part + per_chunk * std::max(G.C_max, 1)) + 16;
  }
  CKC(dev_alloc(c, &c->head_done, (size_t)L * B * Hkv));
  {
    const unsigned long long r_text = B * (unsigned long long)G.text_seq_stride / d, r_anchor = B * (unsigned long long)G.anchor_seq_stride / d,
                             r_pool = B * (unsigned long long)G.pool_seq_stride / d, r_fixed = B * (unsigned long long)G.fixed_seq_stride / d,
                             r_stage = (unsigned long long)Hkv * 2 * G.T_a_pad;
    if (std::max({r_text, r_anchor, r_pool, r_fixed}) >= (1ull << 31)) return fail(WNW_ERR_UNSUPPORTED);  // rows are 32-bit TMA coordinates
    bool ok = encode_store_map(&c->maps_decode.text, cv.text, r_text, d);
    ok = ok && encode_store_map(&c->maps_decode.anchor, cv.anchor, r_anchor, d);
    if (G.kv8 && r_pool) ok = ok && encode_store_map_e4m3(&c->maps_decode.pool, cv.pool, r_pool);
    else ok = ok && encode_store_map(&c->maps_decode.pool, r_pool ? (void *)cv.pool : (void *)cv.text, r_pool ? r_pool : r_text, d);
    ok = ok && encode_store_map(&c->maps_decode.fixed, r_fixed ? (void *)cv.fixed : (void *)cv.text, r_fixed ? r_fixed : r_text, d);
    c->maps_prefill = c->maps_decode;
    ok = ok && encode_store_map(&c->maps_prefill.anchor, c->stage, r_stage, d);
    if (!ok) return fail(WNW_ERR_CUDA);
  }
  c->seqs.assign(B, SeqHost{});
  c->mirror_ptrs.assign(B, nullptr);
  for (auto &sd : c->side) CKE(cudaStreamCreateWithFlags(&sd, cudaStreamNonBlocking));

  c->ev_layer_done.resize(L); c->ev_side_done.resize(L); c->side_recorded.assign(L, 0);
  c->ev_layer_done_cap.resize(L); c->ev_side_done_cap.resize(L);
  for (int l = 0; l < L; ++l) {
    CKE(cudaEventCreateWithFlags(&c->ev_layer_done[l], cudaEventDisableTiming));
    CKE(cudaEventCreateWithFlags(&c->ev_side_done[l], cudaEventDisableTiming));
    CKE(cudaEventCreateWithFlags(&c->ev_layer_done_cap[l], cudaEventDisableTiming));
    CKE(cudaEventCreateWithFlags(&c->ev_side_done_cap[l], cudaEventDisableTiming));
    if (l == 0) {
      CKE(cudaEventCreateWithFlags(&c->ev_sel_fork, cudaEventDisableTiming));
      CKE(cudaEventCreateWithFlags(&c->ev_sel_join, cudaEventDisableTiming));
    }
  }
  CKE(cudaEventCreateWithFlags(&c->ev_place, cudaEventDisableTiming));
  CKE(cudaEventCreateWithFlags(&c->ev_step, cudaEventDisableTiming));
  CKE(cudaEventCreateWithFlags(&c->ev_graph_done, cudaEventDisableTiming));
  CKE(cudaEventCreateWithFlags(&c->ev_recall_all, cudaEventDisableTiming));
  CKC(dev_alloc(c, &c->d_recall_epoch, (size_t)L));
  CKC(dev_alloc(c, &c->d_recall_ctr, (size_t)L));
  CKC(dev_alloc(c, &c->d_step_epoch, 1));
  CKC(dev_alloc(c, &c->d_fold_ctr, 1));
  CKC(dev_alloc(c, &c->d_empty_ctr, (size_t)L));
  if (!full) {
    std::vector<SelectArgs> sel_args(L);
    std::vector<int4> sel_map;
    c->select_single_ok = !c->cv.scope_global;
    for (int l = 0; l < L; ++l) {
      sel_args[l] = static_select_args(c, l);
      c->sel_all_smem = std::max(c->sel_all_smem, c->sel_smem[l]);
      for (int u = 0; u < c->layers[l].upd_count; ++u)   // a layer that ranks by another layer's scores needs them complete
        if (c->layers[c->upd_list[c->layers[l].upd_first + u]].src != l) c->select_single_ok = false;
    }
    auto add = [&](int (&range)[2], auto pred) {
      range[0] = (int)sel_map.size();
      for (int l = 0; l < L; ++l)
        if (pred(c->layers[l])) {
          const int g = select_groups(c->layers[l]);
          for (int y = 0; y < g; ++y) sel_map.push_back(make_int4(l, y, g, 0));
        }
      range[1] = (int)sel_map.size() - range[0];
    };
    add(c->sel_map_single, [](const LayerInfo &li) { return li.n_anchor > 0 || li.upd_count > 0; });
    add(c->sel_map_update, [](const LayerInfo &li) { return li.upd_count > 0; });
    c->sel_map_score[0] = (int)sel_map.size();
    for (int l = 0; l < L; ++l)
      if (c->layers[l].n_anchor > 0) sel_map.push_back(make_int4(l, 0, 1, 0));
    c->sel_map_score[1] = (int)sel_map.size() - c->sel_map_score[0];
    CKC(dev_upload(c, &c->d_sel_args, sel_args));
    CKC(dev_upload(c, &c->d_sel_map, sel_map));
    c->h_sel_args = sel_args; c->h_sel_map = sel_map;
  }
  for (int l = 0; l < L; ++l)
    if (!full && (c->layers[l].n_anchor > 0 || c->layers[l].upd_count > 0)) {
      ++c->n_side_layers;
      c->n_select_ctas += select_groups(c->layers[l]);
    }
  CKE(cudaDeviceSynchronize());
#undef CKC
#undef CKE
  *out = c;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_destroy(wnw_cache_t *c) {
  if (!c) return WNW_ERR_INVALID_ARG;
  destroy_impl(c);
  return WNW_OK;
}

// ---------------------------------------------------------------------------------------------
// Work lists: split every (sequence, KV head) granule space into CTA-sized items
// ---------------------------------------------------------------------------------------------
// Granules per work item, and whether the layer runs as persistent CTAs over a host-balanced schedule.
//
// Independent layers (the default): consecutive layer kernels overlap, so what counts is the work per launch, not
// the span of one kernel.  One-shot 8-warp CTAs over fat items: at least two granules per warp, the longest head in
// at most 16 pieces, and no more split CTAs than a third of the SMs, so that several layer kernels are resident at
// once.  With many sequences this leaves one CTA per head, which writes its output directly (no partial, no merge);
// the block scheduler and the next layers' CTAs fill the SMs that short heads free early.  Measured against the
// persistent schedule on the batched workloads: 77 % vs 71 % and 85 % vs 82 % of the copy bandwidth.
//
// Layers that wait for one another (chained or serial): the span of one kernel counts.  Little work (fits one wave of
// CTAs): small items (two granules per warp), so nearly every byte is in flight at once and the merge stays short.  Otherwise persistent 4-warp CTAs, two per
// SM, over items sized for about one item per CTA and placed longest-first by the host.
static int granules_per_item(const wnw_cache *c, long long total_granules, int longest_head, int n_heads, bool overlapped,
                             bool *throughput) {
  const int nw = attn_warps(false), min_gpi = nw;
  if (overlapped) {
    *throughput = false;
    const int cap = c->n_sm / 3;
    long long per = std::max<long long>(2 * min_gpi, (longest_head + 15) / 16);
    per = std::max<long long>(per, (total_granules + cap - 1) / cap);
    return (int)((per + nw - 1) / nw * nw);
  }
  // two granules per warp: all of an item's bytes are in flight at once and few partials are left to merge (measured on
  // config 1, chained: 212 us per step; one granule per warp 259 us, three 237 us)
  long long per = std::max<long long>(2 * min_gpi, (longest_head + 31) / 32);
  per = (per + nw - 1) / nw * nw;
  *throughput = (total_granules + per - 1) / per + n_heads > c->n_sm;   // more than one wave: build_throughput_items cuts the work
  return (int)per;
}

// Granules of one head: n_gran its whole virtual key space, work those expected to hold data.
static void head_granules(const wnw_cache *c, int layer, int mode, const SeqHost &s, int h, int *n_gran, int *work) {
  const Geometry &G = c->geo;
  const int role = mode == ATTN_DECODE ? c->roles[layer * G.Hkv + h] : ROLE_ANCHOR;
  int fixed_blocks = s.S_fixed;  // what the head kept at placement; a token-compacted head: the blocks its kept positions fill
  if (!s.fixed_blocks.empty() && s.fixed_blocks[layer * G.Hkv + h] >= 0) fixed_blocks = s.fixed_blocks[layer * G.Hkv + h];
  // a tidal head with a token base: its blocks first, then the table's (all dynamic) slots
  const int tidal_units = s.S + (G.token_base && mode == ATTN_DECODE ? fixed_blocks : 0);
  const int audio = (role == ROLE_ANCHOR ? s.C : role == ROLE_TIDAL ? tidal_units : fixed_blocks) * G.gpc;
  *n_gran = G.n_tg + audio;
  // the dynamic slots of a SEGMENT_LAG table are about half empty and cost nothing then
  *work = G.n_tg + audio - (role == ROLE_TIDAL ? (s.S - s.S_base) * G.gpc / 2 : 0);
}

// Throughput regime (more work than one wave of one-shot CTAs): persistent 4-warp CTAs, two per SM, whose copy pipelines
// run from one work item into the next.  What an item costs beyond its bytes decides the cut: a head that stays whole is
// finished inside its CTA, a piece of a split head also pays a fence and a counter round trip under a loaded memory system
// (measured on 12 layers x 16 sequences x 7500 tokens, chained layers: a CTA with two pieces left 6.5 us after one with a
// single piece of the same size).  So heads are cut as little as the balance allows: for a piece size T a head becomes
// round(work / T) even pieces (at least one), the pieces go longest-first to the least loaded CTA, and T is the candidate
// between 0.3 and three even shares of the launch that gives the shortest longest CTA under that cost model.
static void build_throughput_items(const wnw_cache *c, int layer, int mode, const std::vector<int> &seq_ids,
                                   const std::vector<int> &n_gran, const std::vector<int> &n_work, std::vector<WorkItem> &items,
                                   std::vector<HeadItems> &heads, LayerWork &lw, std::vector<int32_t> &order,
                                   std::vector<int32_t> &ranges) {
  const Geometry &G = c->geo;
  const int nw = attn_warps(true), n_heads = (int)seq_ids.size() * G.Hkv;
  const double cost_whole = 5.0, cost_piece = 16.0;   // fixed cost of an item in granules' worth: finished in the CTA / left as a partial
  const double mean_weight = 1.0;                     // weight of the mean CTA load beside the longest one in the objective
  const int per_sm = attn_persistent_ctas_per_sm(G.g, G.d);   // persistent 4-warp CTAs an SM holds
  double total = 0.0;
  for (int hd = 0; hd < n_heads; ++hd) total += n_work[hd];
  const int P = (int)std::min<double>(per_sm * c->n_sm, std::max(1.0, total / (2.0 * nw)));   // at least two granules per warp and CTA
  const bool may_finish = mode != ATTN_PREFILL;       // the prefill scoring pass leaves partials whatever the cut
  auto pieces_of = [&](int hd, double T) { return std::max(1, (int)std::lround(n_work[hd] / T)); };
  auto makespan = [&](double T, std::vector<std::vector<std::pair<int, int>>> *assign) {
    std::vector<std::pair<double, std::pair<int, int>>> its;   // cost, (head, piece)
    for (int hd = 0; hd < n_heads; ++hd) {
      const int np = pieces_of(hd, T);
      for (int x = 0; x < np; ++x)
        its.push_back({(double)n_work[hd] / np + ((np > 1 || !may_finish) ? cost_piece : cost_whole), {hd, x}});
    }
    std::stable_sort(its.begin(), its.end(), [](const auto &x, const auto &y) { return x.first > y.first; });
    std::vector<double> load(P, 0.0);
    if (assign) assign->assign(P, {});
    for (const auto &e : its) {
      const int cta = (int)(std::min_element(load.begin(), load.end()) - load.begin());
      load[cta] += e.first;
      if (assign) (*assign)[cta].push_back(e.second);
    }
    // the longest CTA bounds the launch; the mean load counts too: while some CTAs sit in item overheads the others can
    // only use the bandwidth they leave if there is work left to overlap, so overhead is never free
    double sum = 0.0;
    for (double x : load) sum += x;
    return *std::max_element(load.begin(), load.end()) + mean_weight * sum / P;
  };
  const double share = std::max(total / P, (double)(4 * nw));
  double best_T = share, best = 1e300;
  for (int k = 6; k <= 60; ++k) {   // T from 0.3 to three shares in steps of 5 %; ties go to the larger T (fewer items)
    const double T = share * k / 20.0, ms = makespan(T, nullptr);
    if (ms <= best) { best = ms; best_T = T; }
  }
  std::vector<std::vector<std::pair<int, int>>> assign;
  makespan(best_T, &assign);
  // items in head order (a head's pieces are consecutive: the merge reads their partials as one run)
  std::vector<int> first_item(n_heads, 0);
  for (int hd = 0; hd < n_heads; ++hd) {
    const int i = hd / G.Hkv, h = hd % G.Hkv, n = n_gran[hd], np = pieces_of(hd, best_T);
    const SeqHost &sq = c->seqs[seq_ids[i]];
    const int role = mode == ATTN_DECODE ? c->roles[layer * G.Hkv + h] : ROLE_ANCHOR;
    const int ridx = mode == ATTN_DECODE ? c->role_idx[layer * G.Hkv + h] : h;
    const int perm = (G.token_base && role == ROLE_TIDAL && !sq.fixed_blocks.empty()) ? std::max(sq.fixed_blocks[layer * G.Hkv + h], 0)
                                                                                     : sq.S_base;
    const HeadItems hi{(int)items.size() - lw.first_item, np};
    first_item[hd] = hi.first;
    for (int x = 0; x < np; ++x)
      items.push_back(WorkItem{i, h, (int)((long long)n * x / np), (int)((long long)n * (x + 1) / np), seq_ids[i], role, ridx,
                               role == ROLE_FIXED ? sq.T_a_fixed : sq.T_a, sq.C, perm, sq.T_t, hi.first, hi.count});
    heads.push_back(hi);
    lw.max_count = std::max(lw.max_count, np);
  }
  lw.n_items = (int)items.size() - lw.first_item;
  lw.order_off = (int)order.size();
  lw.ranges_off = (int)ranges.size();
  int pos = 0, n_ctas = 0;
  for (int cta = 0; cta < P; ++cta) {
    if (assign[cta].empty()) continue;
    ranges.push_back(pos);
    for (const auto &hp : assign[cta]) { order.push_back(first_item[hp.first] + hp.second); ++pos; }
    ++n_ctas;
  }
  ranges.push_back(pos);
  lw.n_ctas = n_ctas;
  lw.packed = mode != ATTN_PREFILL;   // the pipeline runs across a CTA's items (its merge scratch sits behind the stages)
}

// Appends the items of one layer for the given sequences.
static void build_layer_items(const wnw_cache *c, int layer, int mode, const std::vector<int> &seq_ids,
                              std::vector<WorkItem> &items, std::vector<HeadItems> &heads, LayerWork &lw,
                              std::vector<int32_t> &order, std::vector<int32_t> &ranges) {
  const Geometry &G = c->geo;
  // n_gran: the head's whole virtual key space (what the items must cover); n_work: the granules expected to hold data
  // (what the items are sized by): the dynamic slots of a SEGMENT_LAG table are about half empty and cost nothing then
  std::vector<int> n_gran(seq_ids.size() * G.Hkv), n_work(seq_ids.size() * G.Hkv);
  long long total = 0;
  int longest = 0;
  for (size_t i = 0; i < seq_ids.size(); ++i) {
    const SeqHost &s = c->seqs[seq_ids[i]];
    for (int h = 0; h < G.Hkv; ++h) {
      int work = 0;
      head_granules(c, layer, mode, s, h, &n_gran[i * G.Hkv + h], &work);
      n_work[i * G.Hkv + h] = work;
      total += work;
      longest = std::max(longest, work);
    }
  }
  bool throughput = false;
  // the prefill scoring pass is a single launch: nothing overlaps it
  const bool overlapped = mode != ATTN_PREFILL && (c->layer_dependency == WNW_LAYERS_INDEPENDENT ||
                                                  c->layer_dependency == WNW_LAYERS_BATCHED);
  int gpi = granules_per_item(c, total, longest, (int)seq_ids.size() * G.Hkv, overlapped, &throughput);
  // BATCHED layers share one launch: the work of the whole step is cut for one wave of CTAs, long heads into pieces as
  // fat as a pack of short ones, short heads packed whole
  const bool batched = overlapped && !throughput && c->layer_dependency == WNW_LAYERS_BATCHED && c->batched_target > 0 &&
                       attn_xpref_fits(G.g, G.d);
  if (batched) gpi = (c->batched_target + attn_warps(false) - 1) / attn_warps(false) * attn_warps(false);
  // Overlapping layers of a tiered cache whose launch is large but would still come out as one unpacked wave (one one-shot
  // CTA per short head, each alone on its SM: nothing covers its start-up and its merge): two persistent 4-warp CTAs per SM
  // cover one another's instead.  Measured on 12 layers x 16 sequences x 7500 tokens with copies skipped: 0.365 -> 0.340 ms
  // per step.  Launches with more heads than SMs keep the packed one-shot CTAs (batch-32 ragged: 1.06 against 1.12 ms), and
  // so does the full-cache kernel (0.878 against 0.895 ms).
  // (What marks such a launch is about as many heads as SMs, not its size: with 64 heads of 7500 tokens the one-shot CTAs
  // win, 0.70 against 0.58 of the copy bandwidth; with 128 heads of 3000 tokens the persistent ones, 0.62 against 0.55.)
  const bool big_single_wave = overlapped && !batched && mode == ATTN_DECODE && total >= 32ll * c->n_sm &&
                               4 * (long long)seq_ids.size() * G.Hkv >= 3ll * c->n_sm;   // decided once the cut is known
  lw.throughput = throughput;
  lw.first_item = (int)items.size();
  lw.head_items_off = (int)heads.size();
  lw.max_count = 0;
  if (throughput) {
    build_throughput_items(c, layer, mode, seq_ids, n_gran, n_work, items, heads, lw, order, ranges);
    return;
  }
  for (size_t i = 0; i < seq_ids.size(); ++i)
    for (int h = 0; h < G.Hkv; ++h) {
      const int n = n_gran[i * G.Hkv + h];
      const SeqHost &sq = c->seqs[seq_ids[i]];
      const int role = mode == ATTN_DECODE ? c->roles[layer * G.Hkv + h] : ROLE_ANCHOR;
      const int ridx = mode == ATTN_DECODE ? c->role_idx[layer * G.Hkv + h] : h;
      // one-shot CTAs: a short head stays in one CTA, which then writes the output itself (no partial, no merge)
      const int nw_ = n_work[i * G.Hkv + h];
      int n_cta = std::max(1, (nw_ + gpi - 1) / gpi);
      // a short head stays in one CTA: up to 128 granules when layers overlap (work per launch counts), 32 when the
      // kernel's span counts (measured, chained config 1: 298 -> 240 us per step against a threshold of 64)
      if (!throughput && nw_ <= (overlapped ? 2 * c->direct_max_granules : c->direct_max_granules / 2)) n_cta = 1;
      if (batched) {   // long heads in pieces as fat as a CTA of their part of the launch
        const int nwp = attn_warps(false);
        const int tg = role == ROLE_TIDAL ? (c->batched_target_tidal + nwp - 1) / nwp * nwp : gpi;
        n_cta = nw_ <= tg * 3 / 2 ? 1 : (nw_ + tg - 1) / tg;
      }
      HeadItems hi{(int)items.size() - lw.first_item, n_cta};
      for (int x = 0; x < n_cta; ++x) {  // even contiguous ranges
        const int g0 = (int)((long long)n * x / n_cta), g1 = (int)((long long)n * (x + 1) / n_cta);
        // S: the head's leading permanent units: slots of the table, or blocks of a tidal head's token base
        const int perm = (G.token_base && role == ROLE_TIDAL && !sq.fixed_blocks.empty()) ? std::max(sq.fixed_blocks[layer * G.Hkv + h], 0)
                                                                                         : sq.S_base;
        items.push_back(WorkItem{(int)i, h, g0, g1, seq_ids[i], role, ridx, role == ROLE_FIXED ? sq.T_a_fixed : sq.T_a, sq.C, perm, sq.T_t,
                                  hi.first, hi.count});
      }
      heads.push_back(hi);
      lw.max_count = std::max(lw.max_count, hi.count);
    }
  lw.n_items = (int)items.size() - lw.first_item;
  lw.n_ctas = 0;
  lw.packed = false;
  if (big_single_wave && lw.n_items <= c->n_sm) {   // see above: the persistent two-per-SM cut instead
    items.resize(lw.first_item);
    heads.resize(lw.head_items_off);
    lw.throughput = true;
    build_throughput_items(c, layer, mode, seq_ids, n_gran, n_work, items, heads, lw, order, ranges);
    return;
  }
  if (!throughput && overlapped && attn_xpref_fits(G.g, G.d) &&
      (lw.n_items > c->n_sm || batched)) {
    // One-shot CTAs of a launch that has more of them than SMs: heads that fit one CTA are packed several to a CTA
    // (consecutive ones, up to about 512 granules of work: a sequence's short heads), which then keeps its copy pipeline
    // running from one head into the next: the fixed cost of a CTA (launch, first reads, first DRAM round trip) is paid
    // once for the pack.  Pieces of split heads keep a CTA each.  Measured: batch-32 ragged 85 -> 91 % of the copy
    // bandwidth; launches with fewer CTAs than SMs lose parallelism instead (16 x 7500: 80 -> 76 %) and are left alone.
    const int target = batched ? gpi : 512;
    lw.order_off = (int)order.size();
    lw.ranges_off = (int)ranges.size();
    int pos = 0, in_pack = 0, pack_work = 0, n_packs = 0;
    bool any = false;
    auto close_pack = [&]() { if (in_pack > 0) { ++n_packs; in_pack = 0; pack_work = 0; } };
    // BATCHED layers: the heads that read no slot come first and never share a CTA with a tidal head: the launch goes
    // out in two parts, the tidal part (cut finer) behind the other
    for (int pass = 0; pass < (batched ? 3 : 1); ++pass) {   // anchor heads, then fixed heads, then tidal heads
      const int tgt = batched && pass == 2 ? c->batched_target_tidal : target;
      for (size_t hd = (size_t)lw.head_items_off; hd < heads.size(); ++hd) {
        const HeadItems &hi = heads[hd];
        const WorkItem &wi = items[lw.first_item + hi.first];
        if (batched && (wi.role == ROLE_ANCHOR ? 0 : wi.role == ROLE_TIDAL ? 2 : 1) != pass) continue;
        if (hi.count > 1) {   // a split head: every piece alone
          close_pack();
          for (int x = 0; x < hi.count; ++x) { ranges.push_back(pos); order.push_back(hi.first + x); ++pos; ++n_packs; }
          continue;
        }
        const int work = n_work[(size_t)wi.i * G.Hkv + wi.h];
        if (in_pack > 0 && pack_work + work > tgt) close_pack();
        if (in_pack == 0) ranges.push_back(pos);
        else any = true;
        order.push_back(hi.first); ++pos; ++in_pack; pack_work += work;
      }
      close_pack();
      if (pass == 0) lw.n_ctas_anchor = batched ? n_packs : 0;
      if (pass == 1 || !batched) lw.n_ctas_free = batched ? n_packs : 0;
    }
    ranges.push_back(pos);
    if (any || batched) { lw.n_ctas = n_packs; lw.packed = true; }
    else { order.resize(lw.order_off); ranges.resize(lw.ranges_off); }
  }
}

static wnw_status_t ensure_worklists(wnw_cache *c) {
  std::vector<int> T_a(c->active.size());
  for (size_t i = 0; i < c->active.size(); ++i) T_a[i] = c->seqs[c->active[i]].T_a;
  if (c->wl_active == c->active && c->wl_T_a == T_a && !c->wl_layers.empty()) return WNW_OK;
  const Geometry &G = c->geo;
  const int mode = c->cfg.mode == WNW_MODE_FULL ? ATTN_FULL : ATTN_DECODE;
  std::vector<WorkItem> items;
  std::vector<HeadItems> heads;
  std::vector<int32_t> order, ranges;
  c->wl_layers.assign(G.L, LayerWork{});
  c->batched_target = 0;
  if (c->layer_dependency == WNW_LAYERS_BATCHED) {   // the step's whole work over one wave of CTAs
    long long total = 0, total_tidal = 0;
    for (int l = 0; l < G.L; ++l)
      for (int b : c->active)
        for (int h = 0; h < G.Hkv; ++h) {
          int n = 0, work = 0;
          head_granules(c, l, mode, c->seqs[b], h, &n, &work);
          if (mode == ATTN_DECODE && c->roles[l * G.Hkv + h] == ROLE_TIDAL) total_tidal += work;
          else total += work;
        }
    // 1.4 x the mean share of an SM: heads are packed whole, so CTAs come out uneven; with this margin the launch stays
    // within one wave (measured, config 1: 57 us per step at 1.2 to 1.7 x the mean, 61 to 65 us at 0.9 and 1.0 x, where
    // a second, nearly empty wave forms, 66 us at 2 x, where too few SMs pull)
    // Tidal heads form a second part of the launch (its CTAs follow those of the first as SMs come free), each cut the same way.
    c->batched_target = (int)std::max<long long>(32, (total * 14 / 10 + c->n_sm - 1) / c->n_sm);
    c->batched_target_tidal = (int)std::max<long long>(32, (total_tidal * 14 / 10 + c->n_sm - 1) / c->n_sm);
    // Where a single layer already fills the machine with CTAs of a decent size its launches stay apart (their steps
    // keep selection and recall inside the step, so nothing would be issued together anyway): the cut of INDEPENDENT.
    if ((total + total_tidal) / G.L > 64ll * c->n_sm) c->batched_target = c->batched_target_tidal = 0;
  }
  if (c->batched_target > 0) {
    // Whole heads and pieces come out uneven: widen the cut until the first part of the launch (the CTAs that read no slot)
    // is at most one wave; a few CTAs beyond it would each add a CTA's whole duration to the step (config 2: 152 CTAs of 184
    // granules 103 us per step, 136 CTAs of 192 granules 75 us).
    for (int attempt = 0; attempt < 12; ++attempt) {
      std::vector<WorkItem> it_t; std::vector<HeadItems> hd_t; std::vector<int32_t> or_t, ra_t;
      int first_part = 0;
      for (int l = 0; l < G.L; ++l) {
        LayerWork lw_t;
        build_layer_items(c, l, mode, c->active, it_t, hd_t, lw_t, or_t, ra_t);
        first_part += lw_t.packed ? lw_t.n_ctas_free : (lw_t.n_ctas > 0 ? lw_t.n_ctas : lw_t.n_items);
      }
      if (first_part <= c->n_sm) break;
      c->batched_target = c->batched_target * 11 / 10 + 1;
    }
  }
  size_t part_total = 0;
  for (int l = 0; l < G.L; ++l) {
    build_layer_items(c, l, mode, c->active, items, heads, c->wl_layers[l], order, ranges);
    c->wl_layers[l].part_off = part_total;
    part_total += (size_t)c->wl_layers[l].n_items;
  }
  // the previous lists may still be read by queued kernels
  CK(cudaDeviceSynchronize());
  if (part_total > c->part_cap_total) {  // one partial region per layer
    float *po = nullptr; float2 *pm = nullptr;
    CK(cudaMalloc((void **)&po, part_total * G.g * G.d * sizeof(float)));
    c->dev_allocs.push_back(po);
    CK(cudaMalloc((void **)&pm, part_total * G.g * sizeof(float2)));
    c->dev_allocs.push_back(pm);
    c->part_o = po; c->part_ml = pm; c->part_cap_total = part_total;
  }
  if (items.size() > c->d_items_cap) {
    CK(cudaMalloc((void **)&c->d_items, items.size() * sizeof(WorkItem)));
    c->dev_allocs.push_back(c->d_items);
    c->d_items_cap = items.size();
  }
  if (heads.size() > c->d_head_items_cap) {
    CK(cudaMalloc((void **)&c->d_head_items, heads.size() * sizeof(HeadItems)));
    c->dev_allocs.push_back(c->d_head_items);
    c->d_head_items_cap = heads.size();
  }
  if (order.size() + ranges.size() > c->d_sched_cap) {
    CK(cudaMalloc((void **)&c->d_sched, (order.size() + ranges.size()) * sizeof(int32_t)));
    c->dev_allocs.push_back(c->d_sched);
    c->d_sched_cap = order.size() + ranges.size();
  }
  if (!order.empty()) {
    CK(cudaMemcpy(c->d_sched, order.data(), order.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    CK(cudaMemcpy(c->d_sched + order.size(), ranges.data(), ranges.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
  }
  c->sched_ranges_base = order.size();
  CK(cudaMemcpy(c->d_items, items.data(), items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice));
  CK(cudaMemcpy(c->d_head_items, heads.data(), heads.size() * sizeof(HeadItems), cudaMemcpyHostToDevice));
  std::vector<int32_t> act(c->active.begin(), c->active.end());
  CK(cudaMemcpy(c->d_active, act.data(), act.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
  c->h_items = items;
  ++c->wl_epoch;
  c->wl_active = c->active;
  c->wl_T_a = T_a;
  return WNW_OK;
}

// ---------------------------------------------------------------------------------------------
// Prefill placement
// ---------------------------------------------------------------------------------------------
extern "C" wnw_status_t wnw_place_prefill(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                          int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_last_dev,
                                          void *cuda_stream) {
  return wnw_place_prefill_multi(c, seq, layer, k_dev, v_dev, n_tokens, audio_begin, audio_end, q_last_dev, 1, cuda_stream);
}

static wnw_status_t place_multi(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_last_dev,
                                int32_t n_queries, void *cuda_stream);

extern "C" wnw_status_t wnw_place_prefill_multi(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                                int32_t n_tokens, int32_t audio_begin, int32_t audio_end,
                                                const void *q_last_dev, int32_t n_queries, void *cuda_stream) {
  // a token-granular base is placed by wnw_place_prefill_tokens only
  if (c && c->geo.token_base) return WNW_ERR_STATE;
  return place_multi(c, seq, layer, k_dev, v_dev, n_tokens, audio_begin, audio_end, q_last_dev, n_queries, cuda_stream);
}

static wnw_status_t place_multi(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                int32_t n_tokens, int32_t audio_begin, int32_t audio_end, const void *q_last_dev,
                                int32_t n_queries, void *cuda_stream) {
  if (!c || !k_dev || !v_dev || n_queries < 1) return WNW_ERR_INVALID_ARG;
  const Geometry &G = c->geo;
  if (seq < 0 || seq >= G.max_batch || layer < 0 || layer >= G.L || n_tokens < 1) return WNW_ERR_INVALID_ARG;
  if (audio_begin < 0 || audio_end < audio_begin || audio_end > n_tokens) return WNW_ERR_INVALID_ARG;
  if (c->in_step) return WNW_ERR_STATE;
  const int T_a = audio_end - audio_begin, T_t = n_tokens - T_a;
  if (T_a > c->cfg.max_audio_tokens || T_t > c->cfg.max_text_tokens) return WNW_ERR_CAPACITY;
  const bool full = c->cfg.mode == WNW_MODE_FULL;
  SeqHost &s = c->seqs[seq];
  if (layer != 0 && (layer != s.placed_layers || T_a != s.T_a || T_t != s.T_t)) return WNW_ERR_STATE;
  const int C_b = (T_a + G.nc - 1) / G.nc, S_b = full ? 0 : slots_total(c->cfg, C_b);
  const int S_base_b = full ? 0 : base_slots_for(c->cfg, C_b);
  if (!full && C_b > 0 && !q_last_dev) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (layer == 0) {
    s.placed_layers = 0;
    const size_t need = full ? 0 : (size_t)mirror_chunks_of(G, C_b) * c->tid_total * 2 * G.ncp * G.d * tidal_elem_bytes(G);
    if (need != s.mirror_bytes) {
      CK(cudaDeviceSynchronize());
      if (s.mirror) cudaFreeHost(s.mirror);
      s.mirror = nullptr; s.mirror_bytes = 0;
      if (need) {
        void *p = nullptr;
        if (cudaHostAlloc(&p, need, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess) {
          cudaGetLastError();
          return WNW_ERR_OOM_HOST;
        }
        if (G.mirror_chunks) memset(p, 0, need);   // chunks that have not arrived yet must read as padding
        void *dp = nullptr;
        CK(cudaHostGetDevicePointer(&dp, p, 0));
        s.mirror = (bf16 *)p; s.mirror_bytes = need;
        c->mirror_ptrs[seq] = (bf16 *)dp;
      } else {
        c->mirror_ptrs[seq] = nullptr;
      }
      CK(cudaMemcpy(c->cv.mirror + seq, &c->mirror_ptrs[seq], sizeof(bf16 *), cudaMemcpyHostToDevice));
    }
    s.T_a = T_a; s.T_t = T_t; s.C = C_b; s.S = S_b; s.S_base = S_base_b;
    s.T_a_fixed = T_a; s.S_fixed = S_base_b; s.append_layer = 0; s.append_n = 0;
    s.fixed_blocks.clear(); s.tok_m.clear();
    c->wl_layers.clear();  // dims may have changed
  }
  // the staging buffer and the partial buffers are shared: order after earlier placements and steps
  if (c->place_recorded) CK(cudaStreamWaitEvent(st, c->ev_place, 0));
  if (c->step_recorded) CK(cudaStreamWaitEvent(st, c->ev_step, 0));
  if (c->recall_all_pending) CK(cudaStreamWaitEvent(st, c->ev_recall_all, 0));
  // chunks start on granule boundaries in every store; the rows between a chunk's last token and the next chunk are zero
  CK(cudaMemsetAsync(c->stage, 0, (size_t)G.Hkv * 2 * G.T_a_pad * G.d * sizeof(bf16), st));
  CK(launch_place_scatter(c->cv, seq, layer, (const bf16 *)k_dev, (const bf16 *)v_dev, n_tokens, audio_begin, audio_end, T_t,
                          C_b, S_b, S_base_b, c->stage, st));
  // e4m3 tidal tier: scales per chunk, and the staged rows of the tidal heads become the values their bytes will decode
  // to, so that the prefill scores below already see what decoding will see
  if (G.kv8 && C_b > 0) CK(launch_quantise_stage(c->cv, seq, layer, c->stage, C_b, st));
  if (!full && C_b > 0) {
    if (c->prefill_seq != seq || c->prefill_T_a != T_a) {
      std::vector<WorkItem> items;
      std::vector<HeadItems> heads;
      LayerWork lw;
      std::vector<int> one{seq};
      std::vector<int32_t> order, ranges;
      build_layer_items(c, layer, ATTN_PREFILL, one, items, heads, lw, order, ranges);
      if (order.size() + ranges.size() > c->pf_sched_cap) {
        CK(cudaMalloc((void **)&c->d_pf_sched, (order.size() + ranges.size()) * sizeof(int32_t)));
        c->dev_allocs.push_back(c->d_pf_sched);
        c->pf_sched_cap = order.size() + ranges.size();
      }
      if (!order.empty()) {
        CK(cudaMemcpyAsync(c->d_pf_sched, order.data(), order.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        CK(cudaMemcpyAsync(c->d_pf_sched + order.size(), ranges.data(), ranges.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
      }
      c->pf_ranges_base = order.size();
      c->pf_n_ctas = lw.n_ctas;
      if ((int)items.size() > c->part_cap_items) return WNW_ERR_CAPACITY;
      if (items.size() > c->pf_items_cap) {
        CK(cudaMalloc((void **)&c->d_pf_items, items.size() * sizeof(WorkItem)));
        c->dev_allocs.push_back(c->d_pf_items);
        c->pf_items_cap = items.size();
      }
      if (!c->d_pf_head_items) {
        CK(cudaMalloc((void **)&c->d_pf_head_items, (size_t)G.Hkv * sizeof(HeadItems)));
        c->dev_allocs.push_back(c->d_pf_head_items);
      }
      for (auto &it : items) it.i = 0;
      CK(cudaMemcpyAsync(c->d_pf_items, items.data(), items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice, st));
      CK(cudaMemcpyAsync(c->d_pf_head_items, heads.data(), heads.size() * sizeof(HeadItems), cudaMemcpyHostToDevice, st));
      CK(cudaStreamSynchronize(st));  // the host vectors go out of scope
      c->pf_n_items = (int)items.size();
      c->pf_throughput = lw.throughput;
      c->h_pf_items = items;
      c->prefill_seq = seq; c->prefill_T_a = T_a;
    }
    AttnArgs a{};
    a.mode = ATTN_PREFILL; a.layer = layer; a.li = c->layers[layer]; a.n_active = 1; a.has_new = 0; a.score_on = 1;
    a.active = c->d_iota + seq; a.items = c->d_pf_items; a.items_host = c->h_pf_items.data(); a.n_items = c->pf_n_items; a.maps = &c->maps_prefill; a.throughput = c->pf_throughput;
    if (c->pf_n_ctas > 0) { a.order = c->d_pf_sched; a.cta_ranges = c->d_pf_sched + c->pf_ranges_base; a.n_ctas = c->pf_n_ctas; }
    a.head_items = c->d_pf_head_items;
    a.anchor_base = c->stage; a.anchor_seq_stride = 0; a.anchor_head0 = 0;
    a.part_o = c->pf_part_o; a.part_ml = c->pf_part_ml; a.gran_em = c->pf_gran_em; a.n_aq = G.Hq; a.n_ag_max = c->n_ag_max;
    for (int qi = 0; qi < n_queries; ++qi) {   // one scoring pass per text query; the scores add up, the last pass places
      a.q = (const bf16 *)q_last_dev + (size_t)qi * G.Hq * G.d;
      CK(launch_attn(c->cv, a, st));
      CK(launch_prefill_select(c->cv, seq, layer, c->d_pf_head_items, c->pf_part_ml, c->pf_gran_em, c->n_ag_max, qi == 0,
                               qi == n_queries - 1, st));
    }
  }
  CK(launch_place_gather(c->cv, seq, layer, full ? 1 : 0, c->stage, C_b, st));
  CK(cudaEventRecord(c->ev_place, st));
  c->place_recorded = true;
  c->last_stream = st;
  s.placed_layers = layer + 1;
  return WNW_OK;
}

static wnw_status_t check_seq_layer(wnw_cache *c, int seq, int layer);
static wnw_status_t drain(wnw_cache *c);

// Streaming audio: n_tokens new audio positions of one layer (layers in order; the grown clip takes effect with the last).
extern "C" wnw_status_t wnw_append_audio(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                         int32_t n_tokens, void *cuda_stream) {
  if (!c || !k_dev || !v_dev || n_tokens < 1) return WNW_ERR_INVALID_ARG;
  const Geometry &G = c->geo;
  if (seq < 0 || seq >= G.max_batch || layer < 0 || layer >= G.L) return WNW_ERR_INVALID_ARG;
  const bool full = c->cfg.mode == WNW_MODE_FULL;
  if (!full && (!c->cfg.streaming_audio || c->cfg.residency != WNW_RESIDENCY_HARD_BUDGET)) return WNW_ERR_UNSUPPORTED;
  if (c->in_step || c->graph_capturing) return WNW_ERR_STATE;
  SeqHost &s = c->seqs[seq];
  if (s.placed_layers != G.L || layer != s.append_layer || (layer > 0 && n_tokens != s.append_n)) return WNW_ERR_STATE;
  if (s.T_a + n_tokens > c->cfg.max_audio_tokens) return WNW_ERR_CAPACITY;
  if (!s.fixed_blocks.empty()) return WNW_ERR_UNSUPPORTED;   // heads compacted token by token have no chunk geometry to grow
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (layer == 0) {   // selections and recalls of earlier steps read and write the tables and slots this touches
    wnw_status_t ds = drain(c);
    if (ds != WNW_OK) return ds;
    CK(cudaStreamSynchronize(st));
    s.append_n = n_tokens;
  }
  const int T_new = s.T_a + n_tokens, C_new = (T_new + G.nc - 1) / G.nc;
  const int S_new = full ? 0 : slots_total(c->cfg, C_new);
  const bool last = layer == G.L - 1;
  CK(launch_append_audio(c->cv, seq, layer, full ? 1 : 0, (const bf16 *)k_dev, (const bf16 *)v_dev, n_tokens, s.T_a, s.S, last ? 1 : 0,
                         T_new, C_new, S_new, st));
  CK(cudaEventRecord(c->ev_place, st));
  c->place_recorded = true;
  c->last_stream = st;
  s.append_layer = last ? 0 : layer + 1;
  if (last) {
    s.T_a = T_new; s.C = C_new; s.S = S_new; s.S_base = S_new;
    c->wl_layers.clear();   // the heads grew: the next step cuts its work anew
    c->prefill_seq = -1;
  }
  return WNW_OK;
}

// Eq. 1 on the host: retention_i = min(s_tilde_i * lambda, 1).
extern "C" wnw_status_t wnw_retention_schedule(const float *s_tilde, int32_t n, float lambda, float *retention) {
  if (!s_tilde || !retention || n < 0 || !(lambda >= 0.f)) return WNW_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!(s_tilde[i] >= 0.f && s_tilde[i] <= 1.f)) return WNW_ERR_INVALID_ARG;
    retention[i] = std::min(s_tilde[i] * lambda, 1.0f);
  }
  return WNW_OK;
}

// positions a head keeps: sum over its segments of floor(retention * length), the arithmetic of the selection kernel
static int kept_positions(int T_a, int seg, float retention) {
  int n = 0;
  for (int lo = 0; lo < T_a; lo += seg) n += (int)std::floor((double)retention * (double)std::min(seg, T_a - lo));
  return n;
}

extern "C" wnw_status_t wnw_place_prefill_tokens(wnw_cache_t *c, int32_t seq, int32_t layer, const void *k_dev, const void *v_dev,
                                                 int32_t n_tokens, int32_t audio_begin, int32_t audio_end,
                                                 const void *q_text_dev, int32_t n_queries, const float *retention,
                                                 int32_t segment_tokens, int32_t variant, void *cuda_stream) {
  if (!c || !retention || segment_tokens < 1 || variant < 0 || variant > 1) return WNW_ERR_INVALID_ARG;
  const Geometry &G = c->geo;
  if (layer < 0 || layer >= G.L || seq < 0 || seq >= G.max_batch) return WNW_ERR_INVALID_ARG;
  if (audio_begin < 0 || audio_end < audio_begin || audio_end > n_tokens) return WNW_ERR_INVALID_ARG;
  const bool full = c->cfg.mode == WNW_MODE_FULL;
  const LayerInfo &li = c->layers[layer];
  const int T_a = audio_end - audio_begin, n_tidal_base = G.token_base ? li.n_tidal : 0;
  const int n_comp = full ? 0 : li.n_fixed + n_tidal_base;   // compressed heads: the fixed ones, then the tidal bases
  if (n_tidal_base > 0 && segment_tokens != G.nc) return WNW_ERR_UNSUPPORTED;   // the quota's segment is the storage segment
  const int tok_cap = G.FB * G.nc;
  const int C_b = (T_a + G.nc - 1) / G.nc, tail_len = T_a - (C_b - 1) * G.nc;
  std::vector<int> blocks(G.Hkv, -1);
  std::vector<int2> m_host(G.Hkv, make_int2(0, 0));
  for (int h = 0; h < G.Hkv && n_comp > 0; ++h) {
    const int role = c->roles[layer * G.Hkv + h];
    if (role != ROLE_FIXED && !(role == ROLE_TIDAL && G.token_base)) continue;
    if (!(retention[h] >= 0.f && retention[h] <= 1.f)) return WNW_ERR_INVALID_ARG;
    const int n = kept_positions(T_a, segment_tokens, retention[h]);
    if (n > tok_cap) return WNW_ERR_CAPACITY;   // the head's compact store holds FB blocks of chunk_tokens rows
    blocks[h] = (n + G.nc - 1) / G.nc;
    if (role == ROLE_TIDAL && T_a > 0)   // the global variant keeps a different number per segment: the device table says
      m_host[h] = variant != 0 ? make_int2(-1, -1)
                               : make_int2((int)std::floor((double)retention[h] * (double)G.nc), (int)std::floor((double)retention[h] * (double)tail_len));
  }
  wnw_status_t rc = place_multi(c, seq, layer, k_dev, v_dev, n_tokens, audio_begin, audio_end, q_text_dev, n_queries, cuda_stream);
  if (rc != WNW_OK || n_comp == 0 || T_a == 0) return rc;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  SeqHost &s = c->seqs[seq];
  if (!c->fixed_tok) {
    int fmax = 0;
    for (const LayerInfo &x : c->layers) fmax = std::max(fmax, (int)x.n_fixed + (G.token_base ? (int)x.n_tidal : 0));
    c->tok_fixed_max = fmax; c->tok_cap = tok_cap;
    c->tok_p_stride = c->cfg.max_audio_tokens;
    const size_t B = G.max_batch;
    if ((rc = dev_alloc(c, &c->tok_work, (size_t)fmax * ((size_t)c->cfg.max_text_tokens + c->cfg.max_audio_tokens))) != WNW_OK) return rc;
    if ((rc = dev_alloc(c, &c->tok_p, (size_t)fmax * c->tok_p_stride)) != WNW_OK) return rc;
    if ((rc = dev_alloc(c, &c->tok_flags, (size_t)fmax * c->tok_p_stride)) != WNW_OK) return rc;
    if ((rc = dev_alloc(c, &c->tok_ret, (size_t)G.Hkv)) != WNW_OK) return rc;
    if ((rc = dev_alloc(c, &c->tok_n, B * std::max(G.F_tot, 1))) != WNW_OK) return rc;
    if ((rc = dev_alloc(c, &c->fixed_tok, B * std::max(G.F_tot, 1) * (size_t)std::max(tok_cap, 1))) != WNW_OK) return rc;
  }
  // the scratch is shared with earlier placements on other streams: the chunk placement above already ordered this
  // stream after them; the retention values travel through a pageable copy, complete on the host side at return
  CK(cudaMemcpyAsync(c->tok_ret, retention, (size_t)G.Hkv * sizeof(float), cudaMemcpyHostToDevice, st));
  if (n_tidal_base > 0)
    CK(cudaMemcpyAsync(c->cv.tok_m + ((size_t)seq * G.L + layer) * G.Hkv, m_host.data(), (size_t)G.Hkv * sizeof(int2),
                       cudaMemcpyHostToDevice, st));
  CK(launch_token_compress(c->cv, seq, layer, n_comp, n_tidal_base, c->stage, (const bf16 *)q_text_dev, n_queries, s.T_t, T_a,
                           segment_tokens, c->tok_ret, variant, c->tok_work, c->tok_p, c->tok_flags, c->tok_p_stride,
                           c->fixed_tok, c->tok_cap, c->tok_n, st));
  CK(cudaEventRecord(c->ev_place, st));
  if (s.fixed_blocks.empty()) s.fixed_blocks.assign((size_t)G.L * G.Hkv, -1);
  if (s.tok_m.empty()) s.tok_m.assign((size_t)G.L * G.Hkv, make_int2(0, 0));
  for (int h = 0; h < G.Hkv; ++h) { s.fixed_blocks[layer * G.Hkv + h] = blocks[h]; s.tok_m[layer * G.Hkv + h] = m_host[h]; }
  c->wl_layers.clear();
  c->tok_last_seq = seq; c->tok_last_layer = layer;
  return WNW_OK;
}

// Index of a head's compact store among the sequence's (fixed heads first, then tidal token bases), -1 if it has none;
// x: its position among the layer's compressed heads.
static int compact_head_of(const wnw_cache *c, int layer, int kv_head, int *x) {
  const int role = c->roles[layer * c->geo.Hkv + kv_head], ridx = c->role_idx[layer * c->geo.Hkv + kv_head];
  const LayerInfo &li = c->layers[layer];
  if (c->cfg.mode != WNW_MODE_TIERED) return -1;
  if (role == ROLE_FIXED) { if (x) *x = ridx; return li.fixed_off + ridx; }
  if (role == ROLE_TIDAL && c->geo.token_base) { if (x) *x = li.n_fixed + ridx; return c->geo.F_fix + li.tid_prefix + ridx; }
  return -1;
}

// per-position prefill scores of one fixed head from the most recent token placement
extern "C" wnw_status_t wnw_get_token_scores(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t kv_head, float *scores,
                                             int32_t capacity) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!scores || kv_head < 0 || kv_head >= c->geo.Hkv) return WNW_ERR_INVALID_ARG;
  int f = 0;
  if (compact_head_of(c, layer, kv_head, &f) < 0) return WNW_ERR_INVALID_ARG;
  if (!c->tok_p || c->tok_last_seq != seq || c->tok_last_layer != layer) return WNW_ERR_STATE;
  const int T_a = c->seqs[seq].T_a;
  if (capacity < T_a) return WNW_ERR_CAPACITY;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  if (T_a > 0) CK(cudaMemcpy(scores, c->tok_p + (size_t)f * c->tok_p_stride, (size_t)T_a * sizeof(float), cudaMemcpyDeviceToHost));
  return WNW_OK;
}

// kept positions (ascending) of a fixed head placed by wnw_place_prefill_tokens
extern "C" wnw_status_t wnw_get_fixed_tokens(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t kv_head, int32_t *positions,
                                             int32_t capacity, int32_t *n) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!positions || !n || kv_head < 0 || kv_head >= c->geo.Hkv) return WNW_ERR_INVALID_ARG;
  const int head = compact_head_of(c, layer, kv_head, nullptr);
  if (head < 0) return WNW_ERR_INVALID_ARG;
  const SeqHost &sq = c->seqs[seq];
  if (!c->fixed_tok || sq.fixed_blocks.empty() || sq.fixed_blocks[layer * c->geo.Hkv + kv_head] < 0) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const size_t fh = (size_t)seq * c->geo.F_tot + head;
  int32_t cnt = 0;
  CK(cudaMemcpy(&cnt, c->tok_n + fh, sizeof(cnt), cudaMemcpyDeviceToHost));
  if (cnt > capacity) return WNW_ERR_CAPACITY;
  if (cnt > 0) CK(cudaMemcpy(positions, c->fixed_tok + fh * c->tok_cap, (size_t)cnt * sizeof(int32_t), cudaMemcpyDeviceToHost));
  *n = cnt;
  return WNW_OK;
}

// One selection launch for the map entries [range[0], range[0] + range[1]); small stacks carry the layers' arguments in
// the kernel parameters.
static cudaError_t select_all(wnw_cache *c, const int *range, const SelectArgs &stp, cudaStream_t st) {
  if (c->geo.L <= SELECT_TABLE_LAYERS && range[1] <= SELECT_TABLE_ENTRIES && !c->h_sel_args.empty())
    return launch_select_all_params(c->cv, c->h_sel_args.data(), c->geo.L, c->h_sel_map.data() + range[0], range[1], stp,
                                    c->sel_all_smem, st);
  return launch_select_all(c->cv, c->d_sel_args, c->d_sel_map + range[0], range[1], stp, c->sel_all_smem, st);
}

// The selection work of a captured step in one launch (two when a layer ranks by another layer's scores).  overlapped:
// it runs beside the step's tidal attention and leaves the step's bookkeeping to a step-end kernel.
static wnw_status_t launch_step_selection(wnw_cache *c, bool overlapped, cudaStream_t st) {
  SelectArgs stp{};
  stp.n_active = (int)c->active.size(); stp.active = c->d_active;
  stp.epoch_words = c->d_recall_epoch; stp.empty_ctr = c->d_empty_ctr; stp.step_epoch = c->d_step_epoch;
  stp.overlapped = overlapped ? 1 : 0;
  if (!c->select_single_ok) {   // first every anchor layer's scores, then every table update
    stp.do_score = 1; stp.do_update = 0;
    CK(select_all(c, c->sel_map_score, stp, st));
    if (c->sel_map_score[1] > 0) c->count_launch(1, 1, true);
  }
  const int *range = c->select_single_ok ? c->sel_map_single : c->sel_map_update;
  stp.do_score = c->select_single_ok ? 1 : 0; stp.do_update = 1;
  if (!overlapped) {
    stp.fold_total = range[1] * stp.n_active; stp.fold_appended = c->appended == 1;
    stp.fold_counter = c->d_fold_ctr; stp.fold_bump_epoch = c->d_step_epoch;
  }
  CK(select_all(c, range, stp, st));
  c->count_launch(1, 1, true);
  return WNW_OK;
}

// ---------------------------------------------------------------------------------------------
// Decode step
// ---------------------------------------------------------------------------------------------
extern "C" wnw_status_t wnw_step_begin(wnw_cache_t *c, const int32_t *active, int32_t n_active) {
  if (!c || !active || n_active < 1 || n_active > c->geo.max_batch) return WNW_ERR_INVALID_ARG;
  if (c->in_step) return WNW_ERR_STATE;
  for (int i = 0; i < n_active; ++i) {
    if (active[i] < 0 || active[i] >= c->geo.max_batch) return WNW_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (active[j] == active[i]) return WNW_ERR_INVALID_ARG;
    if (c->seqs[active[i]].placed_layers != c->geo.L || c->seqs[active[i]].append_layer != 0) return WNW_ERR_STATE;
  }
  DeviceGuard guard(c->cfg.device);
  std::vector<int> want(active, active + n_active);
  if (c->graph_capturing && want != c->graph_prepared) return WNW_ERR_STATE;  // not the set the capture was prepared for
  c->active = want;
  wnw_status_t s = ensure_worklists(c);
  if (s != WNW_OK) return s;
  c->in_step = true; c->next_layer = 0; c->appended = -1;
  for (int &ls : c->last_side_layer) ls = -1;
  return WNW_OK;
}

static bool stream_is_capturing(cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return false; }
  return cs != cudaStreamCaptureStatusNone;
}

// What a layer's selection kernel needs that never changes: the layer, its anchor q-heads, its update list.
static SelectArgs static_select_args(const wnw_cache *c, int layer) {
  const Geometry &G = c->geo;
  const LayerInfo &li = c->layers[layer];
  SelectArgs sa{};
  sa.layer = layer; sa.li = li; sa.active = c->d_active;
  sa.score_on = c->cfg.mode == WNW_MODE_TIERED && li.n_anchor > 0;
  sa.do_score = 1; sa.do_update = 1;
  sa.gran_em = c->gran_em + (size_t)layer * c->gran_em_layer_stride;
  sa.head_mz = c->head_mz + (size_t)layer * G.max_batch * G.Hq;
  sa.n_aq = std::max(li.n_anchor * G.g, 1); sa.n_ag_max = c->n_ag_max;
  int aq = 0;
  for (int h = 0; h < G.Hkv; ++h)
    if (c->roles[layer * G.Hkv + h] == ROLE_ANCHOR)
      for (int r = 0; r < G.g; ++r) sa.aq_head[aq++] = (uint8_t)(h * G.g + r);
  for (int u = 0; u < li.upd_count && u < MAX_UPD_BY_VALUE; ++u) {
    sa.upd_layer[u] = (int16_t)c->upd_list[li.upd_first + u];
    sa.upd_src[u] = (int16_t)c->layers[sa.upd_layer[u]].src;
  }
  return sa;
}

// Decided once per step, at its first layer: how a captured step issues its selection, recall and attention launches.
static void plan_step(wnw_cache *c, bool capturing, bool tiered) {
  const Geometry &G = c->geo;
  // Replayed steps of small launches take their recall out of the captured graph, so that it can overlap the next
  // replay.  Where a launch could fill the machine, its attention CTAs would sit on their SMs while they wait for
  // it, so recall stays inside the step there.
  bool small = true;   // no launch can fill the machine with CTAs that wait
  for (const LayerWork &w : c->wl_layers) small = small && !w.throughput && (w.n_ctas > 0 ? w.n_ctas : w.n_items) <= c->n_sm / 2;
  // the selection kernel of the last layer starts after every attention kernel of the step has completed, so the
  // selection CTA that finishes last in the step may update what those kernels read
  const LayerInfo &last = c->layers[G.L - 1];
  c->cap_fold = capturing && c->graph_capturing && tiered && c->cfg.recall_mode != WNW_RECALL_INLINE &&
                (last.n_anchor > 0 || last.upd_count > 0);
  c->cap_select_all = false;
  c->cap_external_recall = capturing && c->graph_capturing && tiered && c->cfg.recall_mode != WNW_RECALL_INLINE &&
                           small;
  // With the recall outside the graph nothing inside it needs a layer's selection before the step ends: all of it
  // goes into one launch (or two) behind the last attention kernel.
  c->cap_select_all = c->cap_external_recall && small &&
                      (c->select_single_ok ? c->sel_map_single[1] : c->sel_map_update[1]) > 0;
  if (c->cap_select_all) c->cap_fold = true;
  // BATCHED layers: one launch for the whole step where nothing inside the step needs a layer's result earlier
  bool one_shot = G.L <= MULTI_LAYERS_MAX;
  for (const LayerWork &w : c->wl_layers) one_shot = one_shot && !w.throughput;
  c->cap_batched = c->layer_dependency == WNW_LAYERS_BATCHED && c->batched_target > 0 && capturing && c->graph_capturing &&
                   one_shot && (!tiered || c->cap_select_all);
  if (c->cap_batched) c->batch_args.assign(G.L, AttnArgs{});
  // Two parts (slot-free CTAs, then the tidal heads'): every anchor head is in the first, so the step's selection can
  // run beside the second; the step's bookkeeping then waits for both (a step-end kernel instead of the fold).
  c->cap_sel_overlap = false;
  if (c->cap_batched && tiered && c->cap_external_recall && c->cap_select_all) {
    bool any_free = false, any_tidal = false;
    for (const LayerWork &w : c->wl_layers) {
      const int n_free = w.packed ? w.n_ctas_free : 0;
      any_free = any_free || n_free > 0;
      any_tidal = any_tidal || n_free < (w.n_ctas > 0 ? w.n_ctas : w.n_items);
    }
    c->cap_sel_overlap = any_free && any_tidal;
    if (c->cap_sel_overlap) c->cap_fold = false;
  }
}

// An eager layer waits for what earlier work on other streams has to have finished: placements, the recall launch that
// followed the last replayed step, and the previous step's side-stream work on this layer's partials, table and slots.
static wnw_status_t wait_for_earlier_steps(wnw_cache *c, int layer, bool tiered, cudaStream_t st) {
  if (layer == 0 && c->place_recorded) CK(cudaStreamWaitEvent(st, c->ev_place, 0));
  if (layer == 0 && c->recall_all_pending) {  // the recall launch that followed the last replayed step
    CK(cudaStreamWaitEvent(st, c->ev_recall_all, 0));
    c->recall_all_pending = false;
  }
  // side-stream work of the previous step that this layer depends on must have landed: the selection kernel that
  // read this layer's partial buffers, and the recall that refreshed this layer's slots
  if (tiered && c->cfg.recall_mode != WNW_RECALL_INLINE) {
    if (c->side_recorded[layer]) CK(cudaStreamWaitEvent(st, c->ev_side_done[layer], 0));
    const int x = c->tail_of[layer];
    if (x >= 0 && x != layer && c->side_recorded[x]) CK(cudaStreamWaitEvent(st, c->ev_side_done[x], 0));
  }
  return WNW_OK;
}

// All layers of a captured step issued together (BATCHED), at the step's last layer: one launch, or the anchor heads, the
// fixed heads and the tidal heads in turn with the step's selection forked behind the anchor heads.
static wnw_status_t issue_batched_step(wnw_cache *c, bool tiered, bool capturing, int has_new, cudaStream_t st) {
  const Geometry &G = c->geo;
  // Two parts when the step has tidal heads: first the CTAs that read no slot, one wave of them; then, programmatically
  // dependent, those of the tidal heads, which take the SMs as the first part leaves them.  The recall of the previous
  // step (it runs outside the captured graph, beside this step) has landed by then, so no CTA sits on an SM waiting.
  std::vector<int> zero(G.L, 0), n_anchor(G.L, 0), n_fixed(G.L, 0), n_free(G.L, 0), n_tidal(G.L, 0);
  bool any_free = false, any_tidal = false, any_anchor = false, any_fixed = false;
  for (int l = 0; l < G.L; ++l) {
    const LayerWork &w = c->wl_layers[l];
    const int all = w.n_ctas > 0 ? w.n_ctas : w.n_items;
    n_free[l] = w.packed ? w.n_ctas_free : 0;
    n_anchor[l] = w.packed ? w.n_ctas_anchor : 0;
    n_fixed[l] = n_free[l] - n_anchor[l];
    n_tidal[l] = all - n_free[l];
    any_free = any_free || n_free[l] > 0;
    any_tidal = any_tidal || n_tidal[l] > 0;
    any_anchor = any_anchor || n_anchor[l] > 0;
    any_fixed = any_fixed || n_fixed[l] > 0;
  }
  if (tiered && any_free && any_tidal) {
    // anchor heads first: the step's selection depends on them alone and is forked right behind their launch
    const bool split_anchor = c->cap_sel_overlap && any_anchor && any_fixed;
    int n_launch = 0;
    if (split_anchor) {
      CK(launch_attn_multi(c->cv, c->batch_args.data(), G.L, zero.data(), n_anchor.data(), false, st));
      ++n_launch;
    } else {
      CK(launch_attn_multi(c->cv, c->batch_args.data(), G.L, zero.data(), n_free.data(), false, st));
      ++n_launch;
    }
    if (c->cap_sel_overlap) {
      c->appended = has_new;
      CK(cudaEventRecord(c->ev_sel_fork, st));
      CK(cudaStreamWaitEvent(c->side[0], c->ev_sel_fork, 0));
      wnw_status_t rs = launch_step_selection(c, true, c->side[0]);
      if (rs != WNW_OK) return rs;
      CK(cudaEventRecord(c->ev_sel_join, c->side[0]));
    }
    if (split_anchor) {
      CK(launch_attn_multi(c->cv, c->batch_args.data(), G.L, n_anchor.data(), n_fixed.data(), true, st));
      ++n_launch;
    }
    CK(launch_attn_multi(c->cv, c->batch_args.data(), G.L, n_free.data(), n_tidal.data(), true, st));
    ++n_launch;
    c->count_launch(0, n_launch, capturing);
  } else {
    CK(launch_attn_multi(c->cv, c->batch_args.data(), G.L, nullptr, nullptr, false, st));
    c->count_launch(0, 1, capturing);
  }
  return WNW_OK;
}

// Chunk scores, selection and recall of a layer: on a side stream, overlapping whatever follows on the caller's stream
// (captured steps of small launches do all of it in one or two launches at the end of the step instead; head-sharded
// caches only add up their own scores here).
static wnw_status_t issue_side_work(wnw_cache *c, int layer, bool tiered, bool capturing, int has_new, int n_active, cudaStream_t st) {
  const Geometry &G = c->geo;
  (void)G;
  const LayerInfo &li = c->layers[layer];
  const bool defer = tiered && c->cfg.defer_selection;   // head-sharded serving: scores now, everything else at the step's end
  if (defer && capturing) return WNW_ERR_UNSUPPORTED;
  if (layer == 0) c->scores_exported = c->scores_imported = false;
  const bool side_work = tiered && (defer ? li.n_anchor > 0 : (li.n_anchor > 0 || li.upd_count > 0)) && !c->cap_select_all;
  const bool inline_mode = c->cfg.recall_mode == WNW_RECALL_INLINE;
  cudaEvent_t ev_l = capturing ? c->ev_layer_done_cap[layer] : c->ev_layer_done[layer];
  if (side_work && !inline_mode) CK(cudaEventRecord(ev_l, st));
  if (side_work) {
    SelectArgs sa = static_select_args(c, layer);
    sa.n_active = n_active;
    if (defer) sa.do_update = 0;
    if (c->cap_fold) {
      sa.fold_total = c->n_select_ctas * n_active; sa.fold_appended = has_new; sa.fold_counter = c->d_fold_ctr;
      sa.fold_bump_epoch = c->cap_external_recall ? c->d_step_epoch : nullptr;
    }
    if (c->cap_external_recall && c->cap_fold) {   // the epoch arithmetic relies on the bump coming after every selection
      sa.epoch_words = c->d_recall_epoch; sa.empty_ctr = c->d_empty_ctr; sa.step_epoch = c->d_step_epoch;
    }
    const int si = layer % wnw_cache::N_SIDE;
    cudaStream_t ss = inline_mode ? st : c->side[si];
    cudaEvent_t ev_s = capturing ? c->ev_side_done_cap[layer] : c->ev_side_done[layer];
    if (!inline_mode) {
      CK(cudaStreamWaitEvent(ss, ev_l, 0));
      // a routed layer ranks by scores that an earlier layer's selection kernel wrote, maybe on the other side stream
      for (int u = 0; u < li.upd_count; ++u) {
        const int src = c->layers[c->upd_list[li.upd_first + u]].src;
        if (src >= 0 && src != layer && src % wnw_cache::N_SIDE != si)
          CK(cudaStreamWaitEvent(ss, capturing ? c->ev_side_done_cap[src] : c->ev_side_done[src], 0));
      }
      if (c->cv.scope_global && li.upd_count > 0)  // the global accumulator needs every anchor layer's scores of this step
        for (int al : c->anchor_layers)
          if (al != layer && al % wnw_cache::N_SIDE != si)
            CK(cudaStreamWaitEvent(ss, capturing ? c->ev_side_done_cap[al] : c->ev_side_done[al], 0));
    }
    CK(launch_select(c->cv, sa, c->sel_smem[layer], select_groups(li), ss));
    c->count_launch(1, 1, capturing);
    if (li.upd_count > 0 && !c->cap_external_recall && !defer) {
      CK(launch_recall(c->cv, n_active, c->d_active, c->cv.upd_list + li.upd_first, li.upd_count,
                       c->cfg.recall_mode == WNW_RECALL_SKIP, RecallSignal{nullptr, nullptr, nullptr, 0}, ss));
      c->count_launch(2, 1, capturing);
    }
    if (!inline_mode) {
      CK(cudaEventRecord(ev_s, ss));
      if (!capturing) c->side_recorded[layer] = 1;
      c->last_side_layer[si] = layer;
    }
  }
  return WNW_OK;
}

static wnw_status_t decode_layer_impl(wnw_cache *c, int want_mode, int32_t layer, const void *q, const void *k_new,
                                      const void *v_new, void *out, void *cuda_stream) {
  if (!c || !q || !out || ((k_new == nullptr) != (v_new == nullptr))) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != want_mode) return WNW_ERR_STATE;
  if (!c->in_step || layer != c->next_layer) return WNW_ERR_STATE;
  const int has_new = k_new != nullptr;
  if (c->appended >= 0 && c->appended != has_new) return WNW_ERR_STATE;
  if (has_new)
    for (int b : c->active)
      if (c->seqs[b].T_t + 1 > c->cfg.max_text_tokens) return WNW_ERR_CAPACITY;
  const Geometry &G = c->geo;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int n_active = (int)c->active.size();
  const bool tiered = want_mode == WNW_MODE_TIERED;
  // Inside a stream capture the step is one graph: cross-step ordering comes from the join in wnw_step_end, and
  // events recorded outside the capture must not be waited on.
  const bool capturing = stream_is_capturing(st);
  if (layer == 0) c->step_capturing = capturing;
  else if (capturing != c->step_capturing) return WNW_ERR_STATE;
  if (layer == 0) plan_step(c, capturing, tiered);
  if (!capturing) {
    wnw_status_t ws = wait_for_earlier_steps(c, layer, tiered, st);
    if (ws != WNW_OK) return ws;
  }
  const LayerWork &lw = c->wl_layers[layer];
  const LayerInfo &li = c->layers[layer];
  float2 *gran_em_l = c->gran_em + (size_t)layer * c->gran_em_layer_stride;
  float2 *head_mz_l = c->head_mz + (size_t)layer * G.max_batch * G.Hq;
  AttnArgs a{};
  a.mode = tiered ? ATTN_DECODE : ATTN_FULL; a.layer = layer; a.li = li; a.n_active = n_active; a.has_new = has_new;
  a.score_on = tiered && li.n_anchor > 0;
  a.active = c->d_active; a.items = c->d_items + lw.first_item; a.items_host = c->h_items.data() + lw.first_item;
  a.n_items = lw.n_items; a.maps = &c->maps_decode; a.throughput = lw.throughput;
  if (lw.n_ctas > 0) {
    a.order = c->d_sched + lw.order_off; a.cta_ranges = c->d_sched + c->sched_ranges_base + lw.ranges_off; a.n_ctas = lw.n_ctas;
    a.xpref = lw.packed;
  }
  a.head_items = c->d_head_items + lw.head_items_off;
  a.q = (const bf16 *)q; a.k_new = (const bf16 *)k_new; a.v_new = (const bf16 *)v_new;
  a.head_done = c->head_done + (size_t)layer * G.max_batch * G.Hkv; a.head_mz = head_mz_l; a.out = (bf16 *)out;
  a.anchor_base = c->cv.anchor; a.anchor_seq_stride = G.anchor_seq_stride;
  a.anchor_head0 = tiered ? li.anchor_off : layer * G.Hkv;
  a.part_o = c->part_o + lw.part_off * G.g * G.d; a.part_ml = c->part_ml + lw.part_off * G.g;
  a.gran_em = gran_em_l;
  if (c->cap_external_recall && li.n_tidal > 0) { a.wait_epoch = c->d_recall_epoch + layer; a.expect_epoch = c->d_step_epoch; }
  // overlap with the previous layer's kernel when that is what precedes this launch in the stream
  a.pdl = layer > 0 && c->layer_dependency != WNW_LAYERS_SERIAL;
  a.wait_inputs = a.pdl && c->layer_dependency == WNW_LAYERS_CHAINED;
  a.n_aq = std::max(li.n_anchor * G.g, 1); a.n_ag_max = c->n_ag_max;
  cudaEvent_t t0 = nullptr, t1 = nullptr;
  const bool timing = c->timing && !capturing;
  if (timing) {
    for (cudaEvent_t *e : {&t0, &t1}) {
      if (!c->t_free.empty()) { *e = c->t_free.back(); c->t_free.pop_back(); }
      else CK(cudaEventCreate(e));
    }
    CK(cudaEventRecord(t0, st));
  }
  if (c->cap_batched) {
    c->batch_args[layer] = a;
    if (layer == G.L - 1) {
      wnw_status_t bs = issue_batched_step(c, tiered, capturing, has_new, st);
      if (bs != WNW_OK) return bs;
    }
  } else {
    CK(launch_attn(c->cv, a, st));
    c->count_launch(0, 1, capturing);
  }
  if (timing) {
    CK(cudaEventRecord(t1, st));
    c->t_used.emplace_back(t0, t1);
  }
  {
    wnw_status_t ss = issue_side_work(c, layer, tiered, capturing, has_new, n_active, st);
    if (ss != WNW_OK) return ss;
  }
  c->appended = has_new;
  c->next_layer = layer + 1;
  c->last_stream = st;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_decode_layer(wnw_cache_t *c, int32_t layer, const void *q, const void *k_new, const void *v_new,
                                         void *out, void *cuda_stream) {
  return decode_layer_impl(c, WNW_MODE_TIERED, layer, q, k_new, v_new, out, cuda_stream);
}
extern "C" wnw_status_t wnw_decode_layer_full(wnw_cache_t *c, int32_t layer, const void *q, const void *k_new,
                                              const void *v_new, void *out, void *cuda_stream) {
  return decode_layer_impl(c, WNW_MODE_FULL, layer, q, k_new, v_new, out, cuda_stream);
}

// Head-sharded step: the caller's stream waits for the score kernels of the step's anchor layers (side streams).
static wnw_status_t wait_for_scores(wnw_cache *c, cudaStream_t st) {
  for (int l = 0; l < c->geo.L; ++l)
    if (c->layers[l].n_anchor > 0 && c->side_recorded[l]) CK(cudaStreamWaitEvent(st, c->ev_side_done[l], 0));
  return WNW_OK;
}

static wnw_status_t exchange_copy(wnw_cache *c, void *buf, bool out, void *cuda_stream) {
  if (!c || !buf) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != WNW_MODE_TIERED || !c->cfg.defer_selection) return WNW_ERR_UNSUPPORTED;
  if (!c->in_step || c->next_layer != c->geo.L || (out ? c->scores_exported : !c->scores_exported || c->scores_imported)) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (out) {
    wnw_status_t ws = wait_for_scores(c, st);
    if (ws != WNW_OK) return ws;
  }
  CK(launch_exchange_scores(c->cv, (int)c->active.size(), c->d_active, (float *)buf, out ? 1 : 0, st));
  (out ? c->scores_exported : c->scores_imported) = true;
  c->last_stream = st;
  return WNW_OK;
}
extern "C" wnw_status_t wnw_export_scores(wnw_cache_t *c, void *scores_dev, void *cuda_stream) {
  return exchange_copy(c, scores_dev, true, cuda_stream);
}
extern "C" wnw_status_t wnw_import_scores(wnw_cache_t *c, const void *scores_dev, void *cuda_stream) {
  return exchange_copy(c, const_cast<void *>(scores_dev), false, cuda_stream);
}

extern "C" wnw_status_t wnw_export_prefill_tidal(wnw_cache_t *c, int32_t seq, int32_t layer, void *sums_dev, void *cuda_stream) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!sums_dev) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != WNW_MODE_TIERED || !c->cfg.defer_selection) return WNW_ERR_UNSUPPORTED;
  if (c->in_step) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (c->place_recorded) CK(cudaStreamWaitEvent(st, c->ev_place, 0));
  CK(launch_prefill_tidal_sum(c->cv, seq, layer, (float *)sums_dev, st));
  c->last_stream = st;
  return WNW_OK;
}
extern "C" wnw_status_t wnw_import_prefill_tidal(wnw_cache_t *c, int32_t seq, int32_t layer, const void *sums_dev, void *cuda_stream) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!sums_dev) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != WNW_MODE_TIERED || !c->cfg.defer_selection) return WNW_ERR_UNSUPPORTED;
  if (c->in_step) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (c->place_recorded) CK(cudaStreamWaitEvent(st, c->ev_place, 0));
  if (c->layers[layer].n_tidal > 0 && c->seqs[seq].C > 0) CK(launch_prefill_retable(c->cv, seq, layer, (const float *)sums_dev, st));
  CK(cudaEventRecord(c->ev_place, st));
  c->place_recorded = true;
  c->last_stream = st;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_step_end(wnw_cache_t *c, void *cuda_stream) {
  if (!c) return WNW_ERR_INVALID_ARG;
  if (!c->in_step || c->next_layer != c->geo.L) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool capturing = stream_is_capturing(st);
  if (capturing != c->step_capturing) return WNW_ERR_STATE;
  if (capturing && c->cfg.recall_mode != WNW_RECALL_INLINE)
    for (int ls : c->last_side_layer)  // join the forked side streams into the graph
      if (ls >= 0) CK(cudaStreamWaitEvent(st, c->ev_side_done_cap[ls], 0));

  if (capturing && c->cap_select_all) {
    if (c->cap_sel_overlap) {   // forked behind the first part of the attention launch: join it
      CK(cudaStreamWaitEvent(st, c->ev_sel_join, 0));
    } else {
      wnw_status_t rs = launch_step_selection(c, false, st);
      if (rs != WNW_OK) return rs;
    }
  }
  if (c->cfg.mode == WNW_MODE_TIERED && c->cfg.defer_selection) {
    // every tidal layer's selection, table update and recall, from the scores as they stand (the sums over all shards
    // once wnw_import_scores has run; the cache's own sums if it holds every head)
    wnw_status_t ws = wait_for_scores(c, st);
    if (ws != WNW_OK) return ws;
    if (c->sel_map_update[1] > 0) {
      SelectArgs stp{};
      stp.n_active = (int)c->active.size(); stp.active = c->d_active; stp.do_score = 0; stp.do_update = 1;
      CK(select_all(c, c->sel_map_update, stp, st));
      c->count_launch(1, 1, false);
      CK(launch_recall(c->cv, (int)c->active.size(), c->d_active, c->cv.upd_list, (int)c->upd_list.size(),
                       c->cfg.recall_mode == WNW_RECALL_SKIP, RecallSignal{nullptr, nullptr, nullptr, 0}, st));
      c->count_launch(2, 1, false);
    }
  }
  if (!(capturing && c->cap_fold)) {
    CK(launch_step_end(c->cv, (int)c->active.size(), c->d_active, c->appended == 1,
                       (capturing && c->cap_external_recall) ? c->d_step_epoch : nullptr, st));
    c->count_launch(3, 1, capturing);
  }
  if (!capturing) {
    CK(cudaEventRecord(c->ev_step, st));
    c->step_recorded = true;
  }
  if (!capturing) {
    for (int b : c->active)
      if (c->appended == 1) c->seqs[b].T_t += 1;
  } else if (c->graph_capturing) {
    c->graph_active = c->active;
    c->graph_appended = c->appended == 1;
  }
  c->in_step = false;
  c->last_stream = st;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_graph_begin(wnw_cache_t *c, const int32_t *active, int32_t n_active, void *cuda_stream) {
  if (!c || !active || n_active < 1 || n_active > c->geo.max_batch) return WNW_ERR_INVALID_ARG;
  if (c->in_step || c->graph_capturing) return WNW_ERR_STATE;
  if (c->cfg.defer_selection) return WNW_ERR_UNSUPPORTED;   // the exchange between the shards is the caller's: eager steps only
  if (!cuda_stream) return WNW_ERR_INVALID_ARG;  // the legacy default stream cannot be captured
  for (int i = 0; i < n_active; ++i) {
    if (active[i] < 0 || active[i] >= c->geo.max_batch) return WNW_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (active[j] == active[i]) return WNW_ERR_INVALID_ARG;
    if (c->seqs[active[i]].placed_layers != c->geo.L) return WNW_ERR_STATE;
  }
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // work lists are built and uploaded now: nothing may allocate or synchronise once the capture has begun
  c->active.assign(active, active + n_active);
  {
    wnw_status_t ws = ensure_worklists(c);
    if (ws != WNW_OK) return ws;
  }
  c->graph_prepared = c->active;
  // everything queued so far must be ordered before the first replay: drain now, the capture cannot wait on it
  for (auto sd : c->side) CK(cudaStreamSynchronize(sd));
  if (c->last_stream != st) CK(cudaStreamSynchronize(c->last_stream));
  CK(cudaStreamSynchronize(st));
  for (long long &x : c->cap_launches) x = 0;
  CK(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
  c->graph_capturing = true;
  c->graph_active.clear();
  return WNW_OK;
}

extern "C" wnw_status_t wnw_graph_end(wnw_cache_t *c, void *cuda_stream) {
  if (!c) return WNW_ERR_INVALID_ARG;
  if (!c->graph_capturing) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  c->graph_capturing = false;
  cudaGraph_t g = nullptr;
  cudaError_t e = cudaStreamEndCapture(st, &g);
  const bool complete = !c->in_step && !c->graph_active.empty();
  c->in_step = false;
  if (e != cudaSuccess || !g) { c->last_cuda = e; cudaGetLastError(); return WNW_ERR_CUDA; }
  if (!complete) { cudaGraphDestroy(g); return WNW_ERR_STATE; }  // the capture must hold exactly one whole step
  if (c->graph_exec) { cudaGraphExecDestroy(c->graph_exec); c->graph_exec = nullptr; }
  if (c->graph) { cudaGraphDestroy(c->graph); c->graph = nullptr; }
  c->graph = g;
  CK(cudaGraphInstantiate(&c->graph_exec, g, 0));
  c->graph_epoch = c->wl_epoch;
  c->graph_external_recall = c->cap_external_recall;
  c->cap_external_recall = false;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_graph_launch(wnw_cache_t *c, void *cuda_stream) {
  if (!c) return WNW_ERR_INVALID_ARG;
  if (!c->graph_exec || c->in_step || c->graph_capturing) return WNW_ERR_STATE;
  for (int b : c->graph_active) {
    if (c->seqs[b].placed_layers != c->geo.L) return WNW_ERR_STATE;
    if (c->graph_appended && c->seqs[b].T_t + 1 > c->cfg.max_text_tokens) return WNW_ERR_CAPACITY;
  }
  if (c->wl_active != c->graph_active || c->wl_layers.empty() || c->wl_epoch != c->graph_epoch)
    return WNW_ERR_STATE;  // the work lists the graph points at were rebuilt or invalidated
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (c->place_recorded) CK(cudaStreamWaitEvent(st, c->ev_place, 0));
  // side-stream work of earlier eager steps touches the tables and slots the graph reads
  for (int l = 0; l < c->geo.L; ++l)
    if (c->side_recorded[l]) { CK(cudaStreamWaitEvent(st, c->ev_side_done[l], 0)); c->side_recorded[l] = 0; }
  CK(cudaGraphLaunch(c->graph_exec, st));
  for (int k = 0; k < 4; ++k) c->launches[k] += c->cap_launches[k];  // the kernels of the captured step
  if (c->graph_external_recall && !c->upd_list.empty()) {
    ++c->host_epoch;
    // This step's recall, for every layer's table at once, outside the graph: it overlaps the next replay, whose tidal
    // CTAs wait on the per-layer epoch words it publishes.
    CK(cudaEventRecord(c->ev_graph_done, st));
    CK(cudaStreamWaitEvent(c->side[0], c->ev_graph_done, 0));
    CK(launch_recall(c->cv, (int)c->graph_active.size(), c->d_active, c->cv.upd_list, (int)c->upd_list.size(),
                     c->cfg.recall_mode == WNW_RECALL_SKIP, RecallSignal{c->d_recall_epoch, c->d_recall_ctr, c->d_empty_ctr, c->host_epoch},
                     c->side[0]));
    c->count_launch(2, 1, false);
    CK(cudaEventRecord(c->ev_recall_all, c->side[0]));
    c->recall_all_pending = true;
  }
  CK(cudaEventRecord(c->ev_step, st));
  c->step_recorded = true;
  for (int b : c->graph_active)
    if (c->graph_appended) c->seqs[b].T_t += 1;
  c->last_stream = st;
  return WNW_OK;
}

// ---------------------------------------------------------------------------------------------
// Inspection
// ---------------------------------------------------------------------------------------------
static wnw_status_t drain(wnw_cache *c) {
  CK(cudaStreamSynchronize(c->last_stream));
  for (auto sd : c->side) CK(cudaStreamSynchronize(sd));
  return WNW_OK;
}

extern "C" wnw_status_t wnw_sync(wnw_cache_t *c) {
  if (!c) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  wnw_status_t s = drain(c);
  if (s != WNW_OK) return s;
  int32_t st = 0;
  CK(cudaMemcpy(&st, c->cv.status, sizeof(st), cudaMemcpyDeviceToHost));
  if (st & STATUS_TIMEOUT) return WNW_ERR_TIMEOUT;   // a bounded device-side wait ran out (sticky)
  return st ? WNW_ERR_DEVICE_CHECK : WNW_OK;
}

extern "C" wnw_status_t wnw_debug_advance_step_epoch(wnw_cache_t *c, int32_t delta) {
  if (!c) return WNW_ERR_INVALID_ARG;
  if (c->in_step || c->graph_capturing) return WNW_ERR_STATE;
  DeviceGuard guard(c->cfg.device);
  wnw_status_t s = drain(c);
  if (s != WNW_OK) return s;
  int32_t v = 0;
  CK(cudaMemcpy(&v, c->d_step_epoch, sizeof(v), cudaMemcpyDeviceToHost));
  v += delta;
  CK(cudaMemcpy(c->d_step_epoch, &v, sizeof(v), cudaMemcpyHostToDevice));
  return WNW_OK;
}

static wnw_status_t check_seq_layer(wnw_cache *c, int seq, int layer) {
  if (!c) return WNW_ERR_INVALID_ARG;
  if (seq < 0 || seq >= c->geo.max_batch || layer < 0 || layer >= c->geo.L) return WNW_ERR_INVALID_ARG;
  if (c->seqs[seq].placed_layers <= layer) return WNW_ERR_STATE;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_seq_dims(wnw_cache_t *c, int32_t seq, int32_t *T_a, int32_t *T_t, int32_t *C, int32_t *S) {
  if (!c || seq < 0 || seq >= c->geo.max_batch || !T_a || !T_t || !C || !S) return WNW_ERR_INVALID_ARG;
  const SeqHost &s = c->seqs[seq];
  if (s.placed_layers == 0) return WNW_ERR_STATE;
  *T_a = s.T_a; *T_t = s.T_t; *C = s.C; *S = s.S;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_chunk_scores(wnw_cache_t *c, int32_t seq, int32_t layer, float *scores, int32_t *n) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!scores || !n) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const int C_b = c->seqs[seq].C;
  if (C_b > 0)
    CK(cudaMemcpy(scores, c->cv.score_sum + ((size_t)seq * c->geo.L + layer) * c->geo.C_max, C_b * sizeof(float),
                  cudaMemcpyDeviceToHost));
  *n = C_b;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_prefill_scores(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t kv_head, float *scores,
                                               int32_t *n) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!scores || !n || kv_head < 0 || kv_head >= c->geo.Hkv) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const int C_b = c->seqs[seq].C;
  if (C_b > 0)
    CK(cudaMemcpy(scores, c->cv.pre + (((size_t)seq * c->geo.L + layer) * c->geo.Hkv + kv_head) * c->geo.C_max,
                  C_b * sizeof(float), cudaMemcpyDeviceToHost));
  *n = C_b;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_selected(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t *sel, int32_t *n_sel) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!sel || !n_sel) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const size_t bl = (size_t)seq * c->geo.L + layer;
  int32_t n = 0;
  CK(cudaMemcpy(&n, c->cv.n_sel + bl, sizeof(n), cudaMemcpyDeviceToHost));
  if (n > 0) CK(cudaMemcpy(sel, c->cv.sel + bl * c->geo.topk, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
  *n_sel = n;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_residency(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t *slot_chunk, int64_t *stamp,
                                          int32_t *n_slots) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!slot_chunk || !n_slots) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const int S_b = c->seqs[seq].S;
  const size_t off = ((size_t)seq * c->geo.L + layer) * std::max(c->geo.S_max, 1);
  long long steps_b = 0;   // the current copy of the table: the one the next step's attention reads
  CK(cudaMemcpy(&steps_b, c->cv.steps + seq, sizeof(steps_b), cudaMemcpyDeviceToHost));
  if (S_b > 0) {
    CK(cudaMemcpy(slot_chunk, c->cv.slot_chunk + slot_table_off(c->geo, (int)(steps_b & 1), (long long)seq * c->geo.L + layer),
                  S_b * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (stamp) CK(cudaMemcpy(stamp, c->cv.stamp + off, S_b * sizeof(int64_t), cudaMemcpyDeviceToHost));
  }
  *n_slots = S_b;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_fixed_set(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t kv_head, int32_t *chunks,
                                          int32_t *n) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!chunks || !n || kv_head < 0 || kv_head >= c->geo.Hkv) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != WNW_MODE_TIERED || c->roles[layer * c->geo.Hkv + kv_head] != ROLE_FIXED) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const SeqHost &sq_ = c->seqs[seq];   // a token-compacted head keeps positions, not chunks: wnw_get_fixed_tokens
  if (!sq_.fixed_blocks.empty() && sq_.fixed_blocks[layer * c->geo.Hkv + kv_head] >= 0) return WNW_ERR_STATE;
  const size_t fh = (size_t)seq * c->geo.F_tot + c->layers[layer].fixed_off + c->role_idx[layer * c->geo.Hkv + kv_head];
  int32_t cnt = 0;
  CK(cudaMemcpy(&cnt, c->cv.fixed_n + fh, sizeof(cnt), cudaMemcpyDeviceToHost));
  if (cnt > 0) CK(cudaMemcpy(chunks, c->cv.fixed_chunks + fh * c->geo.FB, cnt * sizeof(int32_t), cudaMemcpyDeviceToHost));
  *n = cnt;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_slot_kv(wnw_cache_t *c, int32_t seq, int32_t layer, int32_t kv_head, int32_t slot,
                                        int32_t which, void *rows) {
  wnw_status_t s = check_seq_layer(c, seq, layer);
  if (s != WNW_OK) return s;
  if (!rows || kv_head < 0 || kv_head >= c->geo.Hkv || which < 0 || which > 1) return WNW_ERR_INVALID_ARG;
  if (c->cfg.mode != WNW_MODE_TIERED || c->roles[layer * c->geo.Hkv + kv_head] != ROLE_TIDAL) return WNW_ERR_INVALID_ARG;
  if (slot < 0 || slot >= c->seqs[seq].S) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  if ((s = drain(c)) != WNW_OK) return s;
  const int ridx = c->role_idx[layer * c->geo.Hkv + kv_head];
  const long long off = pool_off(c->geo, c->layers[layer], seq, slot, ridx, which);
  if (!c->geo.kv8) {
    CK(cudaMemcpy(rows, c->cv.pool + off, (size_t)c->geo.nc * c->geo.d * sizeof(bf16), cudaMemcpyDeviceToHost));
    return WNW_OK;
  }
  // e4m3 slots: the bytes, the chunk the table names and its scale; decoded here to the bf16 values they stand for
  const Geometry &G = c->geo;
  std::vector<uint8_t> raw((size_t)G.nc * G.d);
  CK(cudaMemcpy(raw.data(), reinterpret_cast<const uint8_t *>(c->cv.pool) + off, raw.size(), cudaMemcpyDeviceToHost));
  int32_t chunk = -1;
  long long steps = 0;
  CK(cudaMemcpy(&steps, c->cv.steps + seq, sizeof(steps), cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(&chunk, c->cv.slot_chunk + slot_table_off(G, (int)(steps & 1), (long long)seq * G.L + layer) + slot, sizeof(chunk),
                cudaMemcpyDeviceToHost));
  int8_t ex = 0;
  if (chunk >= 0)
    CK(cudaMemcpy(&ex, c->cv.kv_exp + kv_exp_off(G, c->cv.tid_total, seq, c->layers[layer].tid_prefix + ridx, chunk) + which, 1,
                  cudaMemcpyDeviceToHost));
  uint16_t *out = static_cast<uint16_t *>(rows);
  for (int r = 0; r < G.nc; ++r)
    for (int e = 0; e < G.d; ++e) {
      const uint8_t byte = raw[(size_t)r * G.d + (e & ~15) + e4m3_store_pos(which, e & 15)];
      const int E = (byte >> 3) & 15, M = byte & 7;
      const float mag = E == 0 ? std::ldexp((float)M, -9) : std::ldexp(1.f + M / 8.f, E - 7);
      const float val = std::ldexp((byte & 0x80) ? -mag : mag, ex);
      uint32_t u;
      memcpy(&u, &val, 4);
      out[(size_t)r * G.d + e] = (uint16_t)(u >> 16);   // exact: three mantissa bits
    }
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_stats(wnw_cache_t *c, wnw_stats_t *out) {
  if (!c || !out) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  wnw_status_t s = drain(c);
  if (s != WNW_OK) return s;
  const Geometry &G = c->geo;
  const size_t B = (size_t)G.max_batch;
  std::vector<unsigned long long> st(B * 4);
  std::vector<long long> steps(B);
  CK(cudaMemcpy(st.data(), c->cv.stats, st.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(steps.data(), c->cv.steps, B * sizeof(long long), cudaMemcpyDeviceToHost));
  std::vector<int32_t> slot_both(2 * B * G.L * std::max(G.S_max, 1)), slot_chunk(B * G.L * std::max(G.S_max, 1)),
      fixed_n(B * std::max(G.F_tot, 1)), fixed_chunks(B * std::max(G.F_tot, 1) * std::max(G.FB, 1));
  CK(cudaMemcpy(slot_both.data(), c->cv.slot_chunk, slot_both.size() * 4, cudaMemcpyDeviceToHost));
  for (size_t b = 0; b < B; ++b)   // every sequence's current copy
    for (int l = 0; l < G.L; ++l)
      for (int j = 0; j < G.S_max; ++j)
        slot_chunk[(b * G.L + l) * G.S_max + j] = slot_both[slot_table_off(G, (int)(steps[b] & 1), (long long)(b * G.L + l)) + j];
  CK(cudaMemcpy(fixed_n.data(), c->cv.fixed_n, fixed_n.size() * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(fixed_chunks.data(), c->cv.fixed_chunks, fixed_chunks.size() * 4, cudaMemcpyDeviceToHost));
  std::vector<int32_t> seg_kept;
  if (G.token_base) {
    seg_kept.resize(B * (size_t)std::max(c->tid_total, 1) * std::max(G.C_max, 1));
    CK(cudaMemcpy(seg_kept.data(), c->cv.seg_kept, seg_kept.size() * 4, cudaMemcpyDeviceToHost));
  }
  wnw_stats_t r{};
  auto len_of = [&](const SeqHost &sq, int ch) { return std::min(G.nc, sq.T_a - ch * G.nc); };
  for (size_t b = 0; b < B; ++b) {
    const SeqHost &sq = c->seqs[b];
    if (sq.placed_layers == 0) continue;
    r.steps += steps[b];
    r.hits += (int64_t)st[b * 4]; r.misses += (int64_t)st[b * 4 + 1]; r.evictions += (int64_t)st[b * 4 + 2];
    r.recall_bytes += (int64_t)st[b * 4 + 3];
    for (int l = 0; l < sq.placed_layers; ++l) {
      const LayerInfo &li = c->layers[l];
      r.full_audio_tokens += (int64_t)G.Hkv * sq.T_a;
      if (c->cfg.mode == WNW_MODE_FULL) { r.resident_audio_tokens += (int64_t)G.Hkv * sq.T_a; continue; }
      r.resident_audio_tokens += (int64_t)li.n_anchor * sq.T_a;
      int64_t res = 0;
      for (int j = 0; j < sq.S; ++j) {
        const int ch = slot_chunk[(b * G.L + l) * std::max(G.S_max, 1) + j];
        if (ch >= 0) res += len_of(sq, ch);
      }
      if (G.token_base) {   // per head: its kept positions plus the complements of the fetched segments
        for (int h = 0; h < G.Hkv; ++h) {
          if (c->roles[l * G.Hkv + h] != ROLE_TIDAL) continue;
          const size_t fh = b * G.F_tot + G.F_fix + li.tid_prefix + c->role_idx[l * G.Hkv + h];
          const int2 m = sq.tok_m.empty() ? make_int2(0, 0) : sq.tok_m[l * G.Hkv + h];
          const size_t sk = (b * (size_t)c->tid_total + li.tid_prefix + c->role_idx[l * G.Hkv + h]) * std::max(G.C_max, 1);
          int64_t mine = 0;
          for (int j = 0; j < fixed_n[fh]; ++j) mine += -fixed_chunks[fh * G.FB + j] - 2;
          for (int j = 0; j < sq.S; ++j) {
            const int ch = slot_chunk[(b * G.L + l) * std::max(G.S_max, 1) + j];
            if (ch >= 0) mine += len_of(sq, ch) - (m.x < 0 ? seg_kept[sk + ch] : ch == sq.C - 1 ? m.y : m.x);
          }
          r.resident_audio_tokens += mine;
          r.host_audio_tokens += sq.T_a - mine;
        }
      } else {
        r.resident_audio_tokens += (int64_t)li.n_tidal * res;
        r.host_audio_tokens += (int64_t)li.n_tidal * (sq.T_a - res);
      }
      for (int f = 0; f < li.n_fixed; ++f) {
        const size_t fh = b * G.F_tot + li.fixed_off + f;
        for (int j = 0; j < fixed_n[fh]; ++j) {   // entries below -1: blocks of a token-compacted head, -(2 + rows)
          const int ch = fixed_chunks[fh * G.FB + j];
          r.resident_audio_tokens += ch < -1 ? -ch - 2 : len_of(sq, ch);
        }
      }
    }
  }
  *out = r;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_base_slots(wnw_cache_t *c, int32_t seq, int32_t *S_base) {
  if (!c || !S_base || seq < 0 || seq >= c->geo.max_batch) return WNW_ERR_INVALID_ARG;
  if (c->seqs[seq].placed_layers == 0) return WNW_ERR_STATE;
  *S_base = c->seqs[seq].S_base;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_launch_counts(wnw_cache_t *c, int64_t *counts) {
  if (!c || !counts) return WNW_ERR_INVALID_ARG;
  for (int k = 0; k < 4; ++k) counts[k] = c->launches[k];
  return WNW_OK;
}

extern "C" wnw_status_t wnw_set_layer_dependency(wnw_cache_t *c, int32_t mode) {
  if (!c || mode < WNW_LAYERS_INDEPENDENT || mode > WNW_LAYERS_BATCHED) return WNW_ERR_INVALID_ARG;
  if (c->in_step || c->graph_capturing) return WNW_ERR_STATE;
  if (mode != c->layer_dependency) c->wl_layers.clear();  // the work items are sized for the mode
  c->layer_dependency = mode;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_set_kernel_timing(wnw_cache_t *c, int32_t enable) {
  if (!c) return WNW_ERR_INVALID_ARG;
  c->timing = enable != 0;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_get_kernel_time(wnw_cache_t *c, float *attn_ms, int32_t *attn_launches) {
  if (!c || !attn_ms || !attn_launches) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(c->cfg.device);
  wnw_status_t s = drain(c);
  if (s != WNW_OK) return s;
  float total = 0.f;
  for (auto &p : c->t_used) {
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, p.first, p.second));
    total += ms;
    c->t_free.push_back(p.first); c->t_free.push_back(p.second);
  }
  *attn_ms = total;
  *attn_launches = (int32_t)c->t_used.size();
  c->t_used.clear();
  return WNW_OK;
}

extern "C" wnw_status_t wnw_measure_host_link(int32_t device, int64_t bytes, int32_t reps, double *memcpy_gbs, double *kernel_gbs) {
  if (bytes < 4096 || reps < 1 || !memcpy_gbs || !kernel_gbs) return WNW_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  bytes = bytes / 16 * 16;
  void *h = nullptr, *d = nullptr, *hd = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaStream_t st = nullptr;
  wnw_status_t rc = WNW_OK;
  float best_copy = 1e30f, best_kernel = 1e30f;
  if (cudaHostAlloc(&h, bytes, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_OOM_HOST; }
  memset(h, 1, bytes);
  if (cudaMalloc(&d, bytes) != cudaSuccess) { cudaGetLastError(); cudaFreeHost(h); return WNW_ERR_OOM_DEVICE; }
  if (cudaHostGetDevicePointer(&hd, h, 0) != cudaSuccess || cudaEventCreate(&e0) != cudaSuccess ||
      cudaEventCreate(&e1) != cudaSuccess || cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) {
    rc = WNW_ERR_CUDA;
  }
  for (int r = 0; rc == WNW_OK && r < reps + 1; ++r) {
    float ms = 0.f;
    cudaEventRecord(e0, st);
    cudaMemcpyAsync(d, h, bytes, cudaMemcpyHostToDevice, st);
    cudaEventRecord(e1, st);
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = WNW_ERR_CUDA; break; }
    if (r > 0) best_copy = std::min(best_copy, ms);
    cudaEventRecord(e0, st);
    if (launch_copy_plan((const uint4 *)hd, (uint4 *)d, bytes / 16, 32, st) != cudaSuccess) { rc = WNW_ERR_CUDA; break; }
    cudaEventRecord(e1, st);
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = WNW_ERR_CUDA; break; }
    if (r > 0) best_kernel = std::min(best_kernel, ms);
  }
  if (rc == WNW_OK) {
    *memcpy_gbs = (double)bytes / (best_copy * 1e-3) / 1e9;
    *kernel_gbs = (double)bytes / (best_kernel * 1e-3) / 1e9;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (st) cudaStreamDestroy(st);
  cudaFree(d);
  cudaFreeHost(h);
  return rc;
}
