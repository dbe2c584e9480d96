// Recall, step bookkeeping and prefill placement kernels (sm_100a).
#include <cuda_fp8.h>

#include "wnw_internal.cuh"
#include "wnw_tail.cuh"

namespace wnw {

// Address of element `off` of a tidal-tier store (slot pool, host mirror): bf16 elements, or single bytes as e4m3.
__device__ __forceinline__ char *tier_ptr(const Geometry &G, bf16 *base, long long off) {
  return reinterpret_cast<char *>(base) + off * tidal_elem_bytes(G);
}

// ------------------------------------------------------------------------------------------------
// Selection (side stream): grid (n_active), one CTA per sequence.  "Decode-Step Score Aggregation" summed per
// chunk, then "Dynamic Chunk Selection" for every layer whose score source is complete with this layer.
// ------------------------------------------------------------------------------------------------
constexpr int SEL_WARPS = 8;
// One CTA: sequence i of the active list, group `grp` of `n_grp` over the layer's update list.
#ifdef WNW_PHASE_STAMPS   // latency studies only (never in the product build): first start and last end of the launch, ns
__device__ unsigned long long g_sel_time[2] = {~0ull, 0ull};
extern "C" int wnw_debug_read_select_time(unsigned long long *host, int reset) {
  int rc = (int)cudaMemcpyFromSymbol(host, g_sel_time, sizeof(g_sel_time));
  if (reset) { const unsigned long long init[2] = {~0ull, 0ull}; rc |= (int)cudaMemcpyToSymbol(g_sel_time, init, sizeof(init)); }
  return rc;
}
__device__ __forceinline__ unsigned long long sel_gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
__device__ unsigned long long g_sel_phase[8];   // per phase: max over CTAs of the time since the CTA's start, ns
extern "C" int wnw_debug_read_select_phases(unsigned long long *host, int reset) {
  int rc = (int)cudaMemcpyFromSymbol(host, g_sel_phase, sizeof(g_sel_phase));
  if (reset) { const unsigned long long z[8] = {0}; rc |= (int)cudaMemcpyToSymbol(g_sel_phase, z, sizeof(z)); }
  return rc;
}
#define SEL_PHASE(k) do { if (threadIdx.x == 0) atomicMax(&g_sel_phase[k], sel_gtime() - sel_t0); } while (0)
#define SEL_PHASE_T0() const unsigned long long sel_t0 = sel_gtime()
#define SEL_STAMP_START() do { if (threadIdx.x == 0) atomicMin(&g_sel_time[0], sel_gtime()); } while (0)
#define SEL_STAMP_END() do { __syncthreads(); if (threadIdx.x == 0) atomicMax(&g_sel_time[1], sel_gtime()); } while (0)
#else
#define SEL_PHASE(k) do { } while (0)
#define SEL_PHASE_T0() do { } while (0)
#define SEL_STAMP_START() do { } while (0)
#define SEL_STAMP_END() do { } while (0)
#endif
__device__ __forceinline__ void select_body(const CacheView &cv, const SelectArgs &a, int smem_total, unsigned char *smem,
                                            int i, int grp, int n_grp) {
  const Geometry &G = cv.geo;
  constexpr int NT = SEL_WARPS * 32;
  const int b = a.active[i];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const LayerInfo &li = a.li;
  SEL_PHASE_T0();
  // per-sequence scalars: one batch of independent loads
  const int C_b = cv.C[b], S_b = cv.S[b], T_a = cv.T_a[b];
  const int epoch_now = a.step_epoch ? *a.step_epoch : 0;   // read here, not on the way out (the step's own bump comes
                                                            // after every selection CTA has finished)
  const long long step_b = a.overlapped ? cv.steps[b]                    // (nothing bumps it before this launch is joined)
                                        : cv.step_snap[(long long)b * G.L + a.layer];   // not cv.steps: an eager step's bookkeeping kernel
                                                                         // follows the attention kernel, not this one
  const int parity = (int)(step_b & 1);   // the copy of the slot tables this step's attention reads; the update writes the other
  const int n_aq = a.n_aq;
  const bool scored = li.n_anchor > 0 && a.score_on && C_b > 0 && a.do_score;
  // shared-memory layout: (M,Z) of the anchor q-heads | this layer's scores | per-warp update workspaces | granule partials
  float2 *mz_s = reinterpret_cast<float2 *>(smem);
  float *sc_s = reinterpret_cast<float *>(smem + ((size_t)n_aq * 8 + 15) / 16 * 16);
  float *glob_s = sc_s + (C_b + 3) / 4 * 4;   // global scope: sum of all anchor layers' scores
  unsigned char *ws0 = reinterpret_cast<unsigned char *>(glob_s) + ((size_t)C_b * 4 + 15) / 16 * 16;
  const size_t ws_bytes = select_ws_bytes(C_b, S_b);
  const int n_upd = a.do_update ? li.upd_count : 0;
  const int n_par = n_upd < SEL_WARPS ? n_upd : SEL_WARPS;
  float2 *em_s = reinterpret_cast<float2 *>(ws0 + (size_t)n_par * ws_bytes);
  const long long em_room = ((long long)smem_total - (long long)(reinterpret_cast<unsigned char *>(em_s) - smem)) / 8;
  int tile_c = 0;
  if (scored) {
    tile_c = (int)(em_room / ((long long)n_aq * G.gpc));
    if (tile_c > C_b) tile_c = C_b;
  }
  __shared__ int s_last;
  // Every CTA passes here exactly once, also on the error path: the last one of the step closes the step.
  auto close_step = [&]() {
    if (a.fold_total <= 0) return;
    __syncthreads();
    if (threadIdx.x == 0) {
      __threadfence();
      const int prev = atomicAdd(a.fold_counter, 1);
      s_last = prev == a.fold_total - 1;
      if (s_last) *a.fold_counter = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int j = threadIdx.x; j < a.n_active; j += NT) {
      const int bj = a.active[j];
      cv.steps[bj] += 1;
      if (a.fold_appended) cv.text_len[bj] += 1;
    }
    if (threadIdx.x == 0 && a.fold_bump_epoch) *a.fold_bump_epoch += 1;
  };
  if (em_room < 0 || (scored && tile_c < 1)) {  // beyond what the host sized the launch for
    if (threadIdx.x == 0) atomicOr(cv.status, STATUS_BAD_TABLE);
    close_step();
    return;
  }
  auto stage_em = [&](int c0, int c1) {
    const int span = (c1 - c0) * G.gpc, ag0 = c0 * G.gpc;
    for (int idx = threadIdx.x; idx < n_aq * span; idx += NT) {
      const int aq = idx / span, ag = ag0 + (idx - aq * span);
      const int cc = ag / G.gpc, gi = ag - cc * G.gpc;   // a granule holds audio iff it starts inside its chunk's tokens
      if (gi * GR < chunk_len(G, T_a, cc)) cp_async_small(em_s + idx, a.gran_em + ((long long)i * n_aq + aq) * a.n_ag_max + ag, 8);
      else em_s[idx] = make_float2(0.f, 0.f);
    }
  };
  auto upd_of = [&](int u, int &lt, int &src) {
    if (u < MAX_UPD_BY_VALUE) { lt = a.upd_layer[u]; src = a.upd_src[u]; }
    else { lt = cv.upd_list[li.upd_first + u]; src = cv.layers[lt].src; }
  };
  // one batch of copies: (M,Z), the first tile of granule partials, the tables of the first round of updates
  if (scored) {
    if (threadIdx.x < n_aq) cp_async_small(mz_s + threadIdx.x, a.head_mz + (long long)i * G.Hq + a.aq_head[threadIdx.x], 8);
    stage_em(0, tile_c);
  }
  // the tables to update are dealt out over the CTAs of the sequence (grid y), then over the warps of a CTA
  const int u_first = grp * n_par + warp, u_step = n_grp * n_par;
  if (warp < n_par && u_first < n_upd) {
    int lt, src;
    upd_of(u_first, lt, src);
    select_stage(cv, b, lt, src, scored && src == a.layer, C_b, S_b, lane, select_ws_at(ws0 + (size_t)warp * ws_bytes, C_b, S_b), parity);
  }
  SEL_PHASE(0);
  cp_async_commit_wait_all();
  __syncthreads();
  SEL_PHASE(1);
  if (scored) {
    // score_sum[c] = sum over anchor q-heads (head order) of (sum over the chunk's granules of e * 2^(m - M)) / Z
    float *dst = cv.score_sum + ((long long)b * G.L + a.layer) * G.C_max;
    for (int c0 = 0; c0 < C_b; c0 += tile_c) {
      const int c1 = c0 + tile_c < C_b ? c0 + tile_c : C_b, span = (c1 - c0) * G.gpc;
      if (c0 > 0) {
        stage_em(c0, c1);
        cp_async_commit_wait_all();
        __syncthreads();
      }
      for (int c = c0 + threadIdx.x; c < c1; c += NT) {
        float total = 0.f;
        for (int aq = 0; aq < n_aq; ++aq) {
          const float2 mz = mz_s[aq];
          const float2 *p = em_s + (size_t)aq * span + (size_t)(c - c0) * G.gpc;
          float sum_h = 0.f;
          for (int gi = 0; gi < G.gpc; ++gi) sum_h += p[gi].x * exp2f(p[gi].y - mz.x);
          total += mz.y > 0.f ? sum_h / mz.y : 0.f;
        }
        if (!(total >= 0.f) || isinf(total)) atomicOr(cv.status, STATUS_NONFINITE);
        dst[c] = total;
        sc_s[c] = total;
      }
      __syncthreads();
    }
  }
  SEL_PHASE(2);
  if (cv.scope_global && n_upd > 0) {
    // Eq. 2 as printed: one accumulator over all anchor layers of the step, added in layer order
    for (int c = threadIdx.x; c < C_b; c += NT) {
      float gsum = 0.f;
      for (int x = 0; x < cv.n_anchor_layers; ++x) {
        const int al = cv.anchor_layers[x];
        gsum += (al == a.layer && scored) ? sc_s[c] : __ldcg(cv.score_sum + ((long long)b * G.L + al) * G.C_max + c);
      }
      glob_s[c] = gsum;
    }
    __syncthreads();
  }
  if (warp < n_par) {
    const SelectWs w = select_ws_at(ws0 + (size_t)warp * ws_bytes, C_b, S_b);
    for (int u = u_first; u < n_upd; u += u_step) {
      int lt, src;
      upd_of(u, lt, src);
      const bool local = (scored && src == a.layer) || src == -2;
      if (u != u_first) {  // later rounds stage their own tables
        __syncwarp();
        select_stage(cv, b, lt, src, local, C_b, S_b, lane, w, parity);
        cp_async_commit_wait_all();
        __syncwarp();
      }
      const float *rank_by = src == -2 ? glob_s : (local ? sc_s : w.sc);
      if (a.overlapped && a.epoch_words) {
        // the previous step's recall may still be reading this layer's plan: wait (bounded) until it has published the
        // layer's epoch; it never waits for anything this kernel does
        if (lane == 0) {
          int seen;
          const long long t0 = clock64();
          for (;;) {
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];\n" : "=r"(seen) : "l"(a.epoch_words + lt) : "memory");
            if (seen >= epoch_now) break;
            if (clock64() - t0 > 2000000000ll) { atomicOr(cv.status, STATUS_TIMEOUT); break; }
          }
        }
        __syncwarp();
      }
      const int n_copies = G.lag_mode ? select_and_update_lag(cv, b, lt, src, C_b, S_b, cv.S_base[b], T_a, step_b, lane, rank_by, w, parity)
                                      : select_and_update(cv, b, lt, src, C_b, S_b, T_a, step_b, lane, rank_by, w, parity);
      if (a.epoch_words && n_copies == 0 && lane == 0) {
        // one sequence: nobody to count; else the sequence whose plan comes in last publishes
        const bool last = a.n_active == 1 || atomicAdd(a.empty_ctr + lt, 1) == a.n_active - 1;
        if (last) {   // nothing to recall for this layer in this step: its slots are current
          if (a.n_active > 1) a.empty_ctr[lt] = 0;
          __threadfence();
          asm volatile("st.release.gpu.global.s32 [%0], %1;\n" ::"l"(a.epoch_words + lt), "r"(epoch_now + 1) : "memory");
        }
      }
    }
  }
  __syncthreads();
  SEL_PHASE(3);
  close_step();
  SEL_PHASE(4);
}

__global__ void __launch_bounds__(SEL_WARPS * 32) wnw_select_kernel(const __grid_constant__ CacheView cv,
                                                                    const __grid_constant__ SelectArgs a, int smem_total) {
  extern __shared__ __align__(16) unsigned char smem[];
  select_body(cv, a, smem_total, smem, blockIdx.x, blockIdx.y, gridDim.y);
}

// The selection work of SEVERAL layers in one launch (captured steps of small launches: a launch costs about a
// microsecond of the step whatever stream it is on, so thirty per-layer launches are replaced by one or two at the end
// of the step).  grid (n_active, entries of `map`): entry y = (layer, group, groups of that layer).  The layer's
// static arguments come from device memory, what changes per step from `step` (only those fields are read from it).
__global__ void __launch_bounds__(SEL_WARPS * 32) wnw_select_all_kernel(const __grid_constant__ CacheView cv,
                                                                        const SelectArgs *__restrict__ layer_args,
                                                                        const int4 *__restrict__ map,
                                                                        const __grid_constant__ SelectArgs step, int smem_total) {
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ SelectArgs a_s;
  SEL_STAMP_START();
  const int4 m = map[blockIdx.y];
  {
    const int *src = reinterpret_cast<const int *>(layer_args + m.x);
    int *dst = reinterpret_cast<int *>(&a_s);
    for (int x = threadIdx.x; x < (int)(sizeof(SelectArgs) / sizeof(int)); x += blockDim.x) dst[x] = src[x];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    a_s.n_active = step.n_active; a_s.active = step.active;
    a_s.do_score = step.do_score; a_s.do_update = step.do_update;
    a_s.fold_total = step.fold_total; a_s.fold_appended = step.fold_appended;
    a_s.fold_counter = step.fold_counter; a_s.fold_bump_epoch = step.fold_bump_epoch;
    a_s.epoch_words = step.epoch_words; a_s.empty_ctr = step.empty_ctr; a_s.step_epoch = step.step_epoch;
    a_s.overlapped = step.overlapped;
  }
  __syncthreads();
  select_body(cv, a_s, smem_total, smem, blockIdx.x, m.y, m.z);
  SEL_STAMP_END();
}

__global__ void __launch_bounds__(SEL_WARPS * 32) wnw_select_all_p_kernel(const __grid_constant__ CacheView cv,
                                                                          const __grid_constant__ SelectAllTable t,
                                                                          const __grid_constant__ SelectArgs step, int smem_total) {
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ SelectArgs a_s;
  SEL_STAMP_START();
  const int4 m = t.map[blockIdx.y];
  {
    const int *src = reinterpret_cast<const int *>(&t.l[m.x]);
    int *dst = reinterpret_cast<int *>(&a_s);
    for (int x = threadIdx.x; x < (int)(sizeof(SelectArgs) / sizeof(int)); x += blockDim.x) dst[x] = src[x];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    a_s.n_active = step.n_active; a_s.active = step.active;
    a_s.do_score = step.do_score; a_s.do_update = step.do_update;
    a_s.fold_total = step.fold_total; a_s.fold_appended = step.fold_appended;
    a_s.fold_counter = step.fold_counter; a_s.fold_bump_epoch = step.fold_bump_epoch;
    a_s.epoch_words = step.epoch_words; a_s.empty_ctr = step.empty_ctr; a_s.step_epoch = step.step_epoch;
    a_s.overlapped = step.overlapped;
  }
  __syncthreads();
  select_body(cv, a_s, smem_total, smem, blockIdx.x, m.y, m.z);
  SEL_STAMP_END();
}

cudaError_t launch_select_all_params(const CacheView &cv, const SelectArgs *layer_args_host, int n_layers, const int4 *map_host,
                                     int n_entries, const SelectArgs &step, size_t smem_bytes, cudaStream_t st) {
  if (n_entries <= 0 || step.n_active <= 0) return cudaSuccess;
  if (n_layers > SELECT_TABLE_LAYERS || n_entries > SELECT_TABLE_ENTRIES) return cudaErrorInvalidValue;
  static_assert(sizeof(SelectAllTable) + sizeof(CacheView) + sizeof(SelectArgs) < 30000, "kernel parameter space");
  SelectAllTable t;
  memset(&t, 0, sizeof(t));
  memcpy(t.map, map_host, sizeof(int4) * n_entries);
  memcpy(t.l, layer_args_host, sizeof(SelectArgs) * n_layers);
  wnw_select_all_p_kernel<<<dim3(step.n_active, n_entries), SEL_WARPS * 32, smem_bytes, st>>>(cv, t, step, (int)smem_bytes);
  return cudaGetLastError();
}

cudaError_t configure_select_kernel() {
  cudaError_t e = cudaFuncSetAttribute(wnw_select_all_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SELECT_SMEM_CAP);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(wnw_select_all_p_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SELECT_SMEM_CAP);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(wnw_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SELECT_SMEM_CAP);
}

cudaError_t launch_select_all(const CacheView &cv, const SelectArgs *layer_args_dev, const int4 *map_dev, int n_entries,
                              const SelectArgs &step, size_t smem_bytes, cudaStream_t st) {
  if (n_entries <= 0 || step.n_active <= 0) return cudaSuccess;
  wnw_select_all_kernel<<<dim3(step.n_active, n_entries), SEL_WARPS * 32, smem_bytes, st>>>(cv, layer_args_dev, map_dev, step,
                                                                                           (int)smem_bytes);
  return cudaGetLastError();
}

cudaError_t launch_select(const CacheView &cv, const SelectArgs &a, size_t smem_bytes, int groups, cudaStream_t st) {
  wnw_select_kernel<<<dim3(a.n_active, groups), SEL_WARPS * 32, smem_bytes, st>>>(cv, a, (int)smem_bytes);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Recall: copies every planned chunk block pinned host -> slot pool.  A NARROW kernel: RECALL_CTAS CTAs in up to
// RECALL_GROUPS groups; group g walks the layers g, g + groups, ... (earlier layers first), every CTA of the group taking
// its stripe of each block, so several layers' transfers are in flight at once.  The host link needs little in flight
// (32 CTAs x 256 threads x four 16-byte loads = 512 KB); CTAs that wait on the link must not sit on the SMs the
// attention kernels need (40 registers, one CTA per SM, fits beside a resident attention CTA).
// With `sig` set (replayed steps, where this kernel runs outside the captured graph and overlaps the next step) the
// CTA that finishes a layer last publishes the layer's recall epoch, which the next step's tidal CTAs acquire.
// ------------------------------------------------------------------------------------------------
constexpr int RECALL_CTAS = 32, RECALL_GROUPS = 8;
__global__ void __launch_bounds__(256, 6) wnw_recall_kernel(const __grid_constant__ CacheView cv, int n_active,
                                                            const int32_t *active, const int32_t *layers, int n_layers,
                                                            int n_groups, int skip_copy, RecallSignal sig) {
  const Geometry &G = cv.geo;
  constexpr int U = 4;
  const int cpg = gridDim.x / n_groups, grp = blockIdx.x / cpg, rank = blockIdx.x - grp * cpg;
  const int stride = cpg * blockDim.x;
  for (int x = grp; x < n_layers; x += n_groups) {
    const int l = layers[x];
    if (sig.epoch_words) {
      // Already published for this step (by the selection kernel: no sequence planned a copy for this layer).  Its
      // plans must not be read then: the next step's selection may be rewriting them by now.
      int seen;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];\n" : "=r"(seen) : "l"(sig.epoch_words + l) : "memory");
      if (seen >= sig.publish_epoch) continue;
    }
    const LayerInfo &li = cv.layers[l];
    const int n = li.n_tidal * 2 * G.ncp * G.d * tidal_elem_bytes(G) / 16;  // 16-byte vectors per chunk block (far below 2^31)
    bool copies = false;                             // uniform over the whole grid: the plans do not change under this kernel
    for (int i = 0; i < n_active; ++i) {
      const int b = active[i];
      const long long bl = (long long)b * G.L + l;
      const int n_plan = cv.n_plan[bl];
      for (int r = 0; r < n_plan && r < G.plan_cap; ++r) {
        const int c = cv.plan[(bl * G.plan_cap + r) * 2], slot = cv.plan[(bl * G.plan_cap + r) * 2 + 1];
        if (rank == 0 && threadIdx.x == 0) atomicAdd(cv.stats + (long long)b * 4 + 3, (unsigned long long)n * 16ull);
        if (skip_copy) continue;
        copies = true;
        if (c < 0 || c >= cv.C[b] || slot < 0 || slot >= cv.S[b]) {
          if (threadIdx.x == 0) atomicOr(cv.status, STATUS_BAD_TABLE);
          continue;
        }
        const uint4 *src = reinterpret_cast<const uint4 *>(tier_ptr(G, cv.mirror[b], mirror_off(G, li, mirror_chunks_of(G, cv.C[b]), c, 0, 0)));
        uint4 *dst = reinterpret_cast<uint4 *>(tier_ptr(G, cv.pool, pool_off(G, li, b, slot, 0, 0)));
        for (int v0 = rank * blockDim.x + threadIdx.x; v0 < n; v0 += stride * U) {
          uint4 t[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int v = v0 + u * stride;
            if (v < n) t[u] = __ldcs(src + v);
          }
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int v = v0 + u * stride;
            if (v < n) dst[v] = t[u];
          }
        }
      }
    }
    if (sig.epoch_words && !copies) {
      // nothing was written for this layer: its epoch goes out at once, without the round of fences and counting
      if (rank == 0 && threadIdx.x == 0) {
        sig.empty_ctr[l] = 0;
        asm volatile("st.release.gpu.global.s32 [%0], %1;\n" ::"l"(sig.epoch_words + l), "r"(sig.publish_epoch) : "memory");
      }
    } else if (sig.epoch_words) {  // completion of this layer's recall: counted per CTA, published by the last one
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) {
        const int prev = atomicAdd(sig.counters + l, 1);
        if (prev == cpg - 1) {
          sig.counters[l] = 0;
          sig.empty_ctr[l] = 0;
          __threadfence();
          asm volatile("st.release.gpu.global.s32 [%0], %1;\n" ::"l"(sig.epoch_words + l), "r"(sig.publish_epoch) : "memory");
        }
      }
    }
  }
}

cudaError_t launch_recall(const CacheView &cv, int n_active, const int32_t *active, const int32_t *layers_dev, int n_layers,
                          int skip_copy, RecallSignal sig, cudaStream_t st) {
  if (n_layers <= 0 || n_active <= 0) return cudaSuccess;
  // A few tables (one short sequence or two): what counts is when the last block lands, and the link's latency grows
  // several times while attention saturates the memory system, so four times the CTAs keep four times the loads in
  // flight (config 1 back to back: 56 -> 53 us per step).  Many tables: the link's rate counts and more CTAs only take
  // SM resources from attention (batch-32 ragged, link-bound: 2.56 -> 2.88 ms per step with the wide launch).
  const int n_groups = RECALL_GROUPS, n_ctas = sig.epoch_words && (long long)n_active * n_layers <= 64 ? 4 * RECALL_CTAS : RECALL_CTAS;
  const int groups = n_layers < n_groups ? n_layers : n_groups;   // few layers: all CTAs on each block
  wnw_recall_kernel<<<n_ctas / groups * groups, 256, 0, st>>>(cv, n_active, active, layers_dev, n_layers, groups, skip_copy, sig);
  return cudaGetLastError();
}

// Plain host-mapped -> device copy with the recall kernel's access pattern (link probe).
__global__ void __launch_bounds__(256) wnw_copy_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, long long n_vec) {
  constexpr int U = 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; v0 < n_vec; v0 += stride * U) {
    uint4 t[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long v = v0 + u * stride;
      if (v < n_vec) t[u] = __ldcs(src + v);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long v = v0 + u * stride;
      if (v < n_vec) dst[v] = t[u];
    }
  }
}
cudaError_t launch_copy_plan(const uint4 *src, uint4 *dst, long long n_vec, int n_ctas, cudaStream_t st) {
  wnw_copy_kernel<<<n_ctas, 256, 0, st>>>(src, dst, n_vec);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Streaming audio: new positions of one layer go to the tiers their heads keep
// ------------------------------------------------------------------------------------------------
// grid (new token, KV head), one thread per 16-byte piece of the K row and of the V row.  Anchor-like heads: the full-audio
// store.  Tidal heads: the host mirror (mapped pinned memory, written from the device) and, if the position's chunk is
// resident, its slot.  Fixed heads: nothing (their subset is final).  The tables need no growth: placement left every
// slot and every chunk entry up to the capacity empty.  The last layer's launch puts the grown dimensions in force.
__global__ void wnw_append_audio_kernel(const __grid_constant__ CacheView cv, int b, int layer, int full_mode, const bf16 *k,
                                        const bf16 *v, int T_a_old, int S_old, int set_dims, int T_a_new, int C_new, int S_new) {
  const Geometry &G = cv.geo;
  const int ppr = G.d / 8, kv = threadIdx.x / ppr, pc = threadIdx.x - kv * ppr;
  const int tok = blockIdx.x, h = blockIdx.y, tau = T_a_old + tok, ci = tau / G.nc, off = tau - ci * G.nc;
  if (set_dims && tok == 0 && h == 0 && threadIdx.x == 0) { cv.T_a[b] = T_a_new; cv.C[b] = C_new; cv.S[b] = S_new; cv.S_base[b] = S_new; }
  if (kv >= 2) return;
  const uint4 val = *reinterpret_cast<const uint4 *>((kv ? v : k) + ((long long)tok * G.Hkv + h) * G.d + pc * 8);
  const int role = full_mode ? ROLE_ANCHOR : cv.roles[layer * G.Hkv + h];
  const LayerInfo li = cv.layers[layer];
  if (role == ROLE_ANCHOR) {
    const int head = full_mode ? layer * G.Hkv + h : li.anchor_off + cv.role_idx[layer * G.Hkv + h];
    *reinterpret_cast<uint4 *>(cv.anchor + anchor_off(G, G.anchor_seq_stride, b, head, kv) + (long long)(ci * G.ncp + off) * G.d + pc * 8) = val;
  } else if (role == ROLE_TIDAL) {
    const int ridx = cv.role_idx[layer * G.Hkv + h];
    *reinterpret_cast<uint4 *>(cv.mirror[b] + mirror_off(G, li, mirror_chunks_of(G, C_new), ci, ridx, kv) + (long long)off * G.d + pc * 8) = val;
    const long long bl = (long long)b * G.L + layer;
    const int32_t *tab = cv.slot_chunk + slot_table_off(G, (int)(cv.steps[b] & 1), bl);   // the table the next step reads
    for (int j = 0; j < S_old; ++j)
      if (tab[j] == ci) {
        *reinterpret_cast<uint4 *>(cv.pool + pool_off(G, li, b, j, ridx, kv) + (long long)off * G.d + pc * 8) = val;
        break;
      }
  }
}
cudaError_t launch_append_audio(const CacheView &cv, int b, int layer, int full_mode, const bf16 *k, const bf16 *v, int n_tokens,
                                int T_a_old, int S_old, int set_dims, int T_a_new, int C_new, int S_new, cudaStream_t st) {
  const int threads = (2 * cv.geo.d / 8 + 31) / 32 * 32;
  wnw_append_audio_kernel<<<dim3((unsigned)n_tokens, (unsigned)cv.geo.Hkv), threads, 0, st>>>(cv, b, layer, full_mode, k, v, T_a_old, S_old,
                                                                                            set_dims, T_a_new, C_new, S_new);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Step bookkeeping
// ------------------------------------------------------------------------------------------------
__global__ void wnw_step_end_kernel(const __grid_constant__ CacheView cv, int n_active, const int32_t *active, int appended,
                                    int32_t *bump_epoch) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0 && bump_epoch) *bump_epoch += 1;  // replayed steps: the recall of this step will publish this epoch
  if (i >= n_active) return;
  const int b = active[i];
  cv.steps[b] += 1;
  if (appended) cv.text_len[b] += 1;
}
cudaError_t launch_step_end(const CacheView &cv, int n_active, const int32_t *active, int appended, int32_t *bump_epoch,
                            cudaStream_t st) {
  wnw_step_end_kernel<<<(n_active + 127) / 128, 128, 0, st>>>(cv, n_active, active, appended, bump_epoch);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Prefill placement ("Prefill Compression", chunk level)
// ------------------------------------------------------------------------------------------------

// Splits one layer's prefill K,V [n_tokens][Hkv][d] into the text store and a per-head staging copy of the audio
// (anchor layout [Hkv][K|V][T_a_pad][d]), zero-pads the staging tail, and resets the layer's tables.
__global__ void __launch_bounds__(256) wnw_place_scatter_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                const bf16 *k, const bf16 *v, int n_tokens, int ab, int ae,
                                                                int T_t, int C_b, int S_b, int S_base, bf16 *stage) {
  const Geometry &G = cv.geo;
  const int T_a = ae - ab, vec_per_row = G.d / 8;
  const long long bl = (long long)b * G.L + layer;
  if (blockIdx.x == 0) {
    if (threadIdx.x == 0) {
      cv.text_len[b] = T_t; cv.T_a[b] = T_a; cv.C[b] = C_b; cv.S[b] = S_b; cv.S_base[b] = S_base;
      cv.n_sel[bl] = 0; cv.n_plan[bl] = 0;
      if (layer == 0) {
        cv.steps[b] = 0;
        for (int x = 0; x < 4; ++x) cv.stats[(long long)b * 4 + x] = 0ull;
      }
    }
    for (int s = threadIdx.x; s < G.S_max; s += blockDim.x) {   // placement resets the step count: copy 0 is current
      cv.slot_chunk[slot_table_off(G, 0, bl) + s] = -1; cv.slot_chunk[slot_table_off(G, 1, bl) + s] = -1; cv.stamp[bl * G.S_max + s] = 0;
    }
    for (int c = threadIdx.x; c < G.C_max; c += blockDim.x) { cv.chunk_slot[bl * G.C_max + c] = -1; cv.score_sum[bl * G.C_max + c] = 0.f; }
    const LayerInfo li = cv.layers[layer];
    for (int f = threadIdx.x; f < li.n_fixed; f += blockDim.x) cv.fixed_n[(long long)b * G.F_tot + li.fixed_off + f] = 0;
  }
  const long long work = (long long)n_tokens * G.Hkv * 2 * vec_per_row;   // the staging copy was zeroed by the caller
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < work; idx += (long long)gridDim.x * blockDim.x) {
    const int vv = (int)(idx % vec_per_row);
    long long t = idx / vec_per_row;
    const int kv = (int)(t % 2); t /= 2;
    const int h = (int)(t % G.Hkv);
    const int tok = (int)(t / G.Hkv);
    const uint4 val = *reinterpret_cast<const uint4 *>((kv ? v : k) + ((long long)tok * G.Hkv + h) * G.d + vv * 8);
    bf16 *dst;
    if (tok >= ab && tok < ae) {  // audio token tau sits in row (tau / nc) * ncp + tau % nc: every chunk starts on a granule
      const int tau = tok - ab, cc = tau / G.nc;
      dst = stage + anchor_off(G, 0, 0, h, kv) + (long long)(cc * G.ncp + (tau - cc * G.nc)) * G.d + vv * 8;
    } else {
      dst = cv.text + text_off(G, b, layer, h, kv) + (long long)(tok < ab ? tok : tok - T_a) * G.d + vv * 8;
    }
    *reinterpret_cast<uint4 *>(dst) = val;
  }
}
cudaError_t launch_place_scatter(const CacheView &cv, int b, int layer, const bf16 *k, const bf16 *v, int n_tokens, int ab,
                                 int ae, int T_t, int C_b, int S_b, int S_base, bf16 *stage, cudaStream_t st) {
  wnw_place_scatter_kernel<<<296, 256, 0, st>>>(cv, b, layer, k, v, n_tokens, ab, ae, T_t, C_b, S_b, S_base, stage);
  return cudaGetLastError();
}

// One CTA.  From the prefill attention partials of q_last: pre[h][c] per non-anchor KV head, then the fixed heads'
// own top-S sets and the tidal heads' shared top-S table (rank r -> slot r, stamp -1-r).
__global__ void __launch_bounds__(512) wnw_prefill_select_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                 const HeadItems *head_items, const float2 *part_ml,
                                                                 const float2 *gran_em, int n_ag_max, int first, int last) {
  extern __shared__ float sm[];  // [Hq] M, [Hq] Z, [C_max] keys (as u64 pairs)
  const Geometry &G = cv.geo;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarp = blockDim.x >> 5;
  const int g = G.g, C_b = cv.C[b], S_b = cv.S_base[b], T_a = cv.T_a[b];   // the prefill placement fills the permanent slots
  float *sM = sm, *sZ = sm + G.Hq;
  unsigned long long *skey = reinterpret_cast<unsigned long long *>(sm + 2 * G.Hq + (2 * G.Hq & 1));
  const LayerInfo li = cv.layers[layer];
  const long long bl = (long long)b * G.L + layer;
  for (int hq = warp; hq < G.Hq; hq += nwarp) {
    const HeadItems hi = head_items[hq / g];
    const int row = hq % g;
    float M = -INFINITY;
    for (int n = lane; n < hi.count; n += 32) M = fmaxf(M, part_ml[(long long)(hi.first + n) * g + row].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float Z = 0.f;
    for (int n = lane; n < hi.count; n += 32) {
      const float2 ml = part_ml[(long long)(hi.first + n) * g + row];
      Z += M > -INFINITY ? ml.y * exp2f(ml.x - M) : 0.f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
    if (lane == 0) { sM[hq] = M; sZ[hq] = Z; }
  }
  __syncthreads();
  float *pre = cv.pre + bl * G.Hkv * G.C_max;
  for (int idx = tid; idx < G.Hkv * C_b; idx += blockDim.x) {
    const int h = idx / C_b, c = idx - h * C_b;
    float total = 0.f;
    if (cv.roles[layer * G.Hkv + h] != ROLE_ANCHOR) {
      for (int r = 0; r < g; ++r) {
        const int hq = h * g + r;
        const float2 *ge = gran_em + (long long)hq * n_ag_max + (long long)c * G.gpc;
        float sum_h = 0.f;
        for (int gi = 0; gi < G.gpc; ++gi) {
          if (gi * GR >= chunk_len(G, T_a, c)) break;
          sum_h += ge[gi].x * exp2f(ge[gi].y - sM[hq]);
        }
        total += sZ[hq] > 0.f ? sum_h / sZ[hq] : 0.f;
      }
    }
    // summed over the text queries, one launch per query ("Prefill Compression": p_prefill = sum over text queries)
    pre[(long long)h * G.C_max + c] = first ? total : pre[(long long)h * G.C_max + c] + total;
  }
  if (!last) return;   // the placement follows the last query
  __syncthreads();
  // fixed heads: rank by counting
  for (int h = 0; h < G.Hkv; ++h) {
    if (cv.roles[layer * G.Hkv + h] != ROLE_FIXED) continue;
    for (int c = tid; c < C_b; c += blockDim.x) skey[c] = rank_key(pre[(long long)h * G.C_max + c], chunk_len(G, T_a, c), c);
    __syncthreads();
    const long long fh = (long long)b * G.F_tot + li.fixed_off + cv.role_idx[layer * G.Hkv + h];
    for (int c = tid; c < C_b; c += blockDim.x) {
      const unsigned long long me = skey[c];
      int rank = 0;
      for (int x = 0; x < C_b; ++x) rank += skey[x] > me;
      if (rank < S_b) cv.fixed_chunks[fh * G.FB + rank] = c;
    }
    if (tid == 0) cv.fixed_n[fh] = S_b;
    __syncthreads();
  }
  if (li.n_tidal > 0) {
    for (int c = tid; c < C_b; c += blockDim.x) {
      float total = 0.f;
      for (int h = 0; h < G.Hkv; ++h)
        if (cv.roles[layer * G.Hkv + h] == ROLE_TIDAL) total += pre[(long long)h * G.C_max + c];
      skey[c] = rank_key(total, chunk_len(G, T_a, c), c);
    }
    __syncthreads();
    for (int c = tid; c < C_b; c += blockDim.x) {
      const unsigned long long me = skey[c];
      int rank = 0;
      for (int x = 0; x < C_b; ++x) rank += skey[x] > me;
      if (rank < S_b) {
        cv.slot_chunk[slot_table_off(G, 0, bl) + rank] = c;
        cv.chunk_slot[bl * G.C_max + c] = rank;
        cv.stamp[bl * G.S_max + rank] = -1 - (long long)rank;
      }
    }
  }
}
// Head-sharded placement.  (1) This cache's share of the tidal ranking of (b, layer): the prefill scores of its own tidal
// heads added in head order, [C_max] floats, zero past the sequence's chunks.
__global__ void wnw_prefill_tidal_sum_kernel(const __grid_constant__ CacheView cv, int b, int layer, float *dst) {
  const Geometry &G = cv.geo;
  const int C_b = cv.C[b];
  const float *pre = cv.pre + ((long long)b * G.L + layer) * G.Hkv * G.C_max;
  for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < G.C_max; c += gridDim.x * blockDim.x) {
    float total = 0.f;
    if (c < C_b)
      for (int h = 0; h < G.Hkv; ++h)
        if (cv.roles[layer * G.Hkv + h] == ROLE_TIDAL) total += pre[(long long)h * G.C_max + c];
    dst[c] = total;
  }
}
// (2) The table of (b, layer) ranked anew from the sums over all shards (rank r -> slot r, stamp -1-r, as at placement)...
__global__ void __launch_bounds__(512) wnw_prefill_retable_kernel(const __grid_constant__ CacheView cv, int b, int layer, const float *sums) {
  extern __shared__ unsigned long long rkey[];
  const Geometry &G = cv.geo;
  const int C_b = cv.C[b], S_b = cv.S_base[b], T_a = cv.T_a[b], tid = threadIdx.x;
  const long long bl = (long long)b * G.L + layer;
  for (int s = tid; s < G.S_max; s += blockDim.x) {
    cv.slot_chunk[slot_table_off(G, 0, bl) + s] = -1; cv.slot_chunk[slot_table_off(G, 1, bl) + s] = -1; cv.stamp[bl * G.S_max + s] = 0;
  }
  for (int c = tid; c < G.C_max; c += blockDim.x) cv.chunk_slot[bl * G.C_max + c] = -1;
  for (int c = tid; c < C_b; c += blockDim.x) rkey[c] = rank_key(sums[c], chunk_len(G, T_a, c), c);
  __syncthreads();
  const int parity = (int)(cv.steps[b] & 1);
  for (int c = tid; c < C_b; c += blockDim.x) {
    const unsigned long long me = rkey[c];
    int rank = 0;
    for (int x = 0; x < C_b; ++x) rank += rkey[x] > me;
    if (rank < S_b) {
      cv.slot_chunk[slot_table_off(G, parity, bl) + rank] = c;
      cv.chunk_slot[bl * G.C_max + c] = rank;
      cv.stamp[bl * G.S_max + rank] = -1 - (long long)rank;
    }
  }
}
// ... (3) and its slots filled from the host mirror: one CTA per slot copies the chunk's block (all tidal heads, K and V).
__global__ void wnw_refill_slots_kernel(const __grid_constant__ CacheView cv, int b, int layer) {
  const Geometry &G = cv.geo;
  const LayerInfo li = cv.layers[layer];
  const long long bl = (long long)b * G.L + layer;
  const int slot = blockIdx.x, c = cv.slot_chunk[slot_table_off(G, (int)(cv.steps[b] & 1), bl) + slot];
  if (c < 0 || li.n_tidal == 0) return;
  const long long n_vec = (long long)li.n_tidal * 2 * G.ncp * G.d * tidal_elem_bytes(G) / 16;
  const uint4 *src = reinterpret_cast<const uint4 *>(tier_ptr(G, cv.mirror[b], mirror_off(G, li, mirror_chunks_of(G, cv.C[b]), c, 0, 0)));
  uint4 *dst = reinterpret_cast<uint4 *>(tier_ptr(G, cv.pool, pool_off(G, li, b, slot, 0, 0)));
  for (long long i = threadIdx.x; i < n_vec; i += blockDim.x) dst[i] = src[i];
}
// Head-sharded step: grid (active sequence, layer).  Out: the cache's own partial sums of the layer's chunk scores, a zero
// row where none of the layer's anchor heads is the cache's own (the row may still hold the sums taken back in an earlier
// step).  In: the sums over all shards.
__global__ void wnw_exchange_scores_kernel(const __grid_constant__ CacheView cv, const int32_t *active, float *buf, int out) {
  const Geometry &G = cv.geo;
  const int i = blockIdx.x, l = blockIdx.y, b = active[i];
  float *mine = cv.score_sum + ((long long)b * G.L + l) * G.C_max, *theirs = buf + ((long long)i * G.L + l) * G.C_max;
  const bool own = cv.layers[l].n_anchor > 0;
  for (int c = threadIdx.x; c < G.C_max; c += blockDim.x) {
    if (out) theirs[c] = own && c < cv.C[b] ? mine[c] : 0.f;
    else mine[c] = theirs[c];
  }
}
cudaError_t launch_exchange_scores(const CacheView &cv, int n_active, const int32_t *active, float *buf, int out, cudaStream_t st) {
  if (cv.geo.C_max < 1) return cudaSuccess;
  wnw_exchange_scores_kernel<<<dim3((unsigned)n_active, (unsigned)cv.geo.L), 128, 0, st>>>(cv, active, buf, out);
  return cudaGetLastError();
}
cudaError_t launch_prefill_tidal_sum(const CacheView &cv, int b, int layer, float *dst, cudaStream_t st) {
  wnw_prefill_tidal_sum_kernel<<<4, 256, 0, st>>>(cv, b, layer, dst);
  return cudaGetLastError();
}
cudaError_t launch_prefill_retable(const CacheView &cv, int b, int layer, const float *sums, cudaStream_t st) {
  wnw_prefill_retable_kernel<<<1, 512, (size_t)std::max(cv.geo.C_max, 1) * 8, st>>>(cv, b, layer, sums);
  if (cv.geo.S_max > 0) wnw_refill_slots_kernel<<<cv.geo.S_max, 256, 0, st>>>(cv, b, layer);
  return cudaGetLastError();
}

cudaError_t launch_prefill_select(const CacheView &cv, int b, int layer, const HeadItems *head_items, const float2 *part_ml,
                                  const float2 *gran_em, int n_ag_max, int first, int last, cudaStream_t st) {
  const size_t smem = (size_t)(2 * cv.geo.Hq + 2) * sizeof(float) + (size_t)cv.geo.C_max * sizeof(unsigned long long);
  wnw_prefill_select_kernel<<<1, 512, smem, st>>>(cv, b, layer, head_items, part_ml, gran_em, n_ag_max, first, last);
  return cudaGetLastError();
}

// grid (C_b, Hkv).  Moves one chunk of one head from staging to its tier: anchor store (anchor heads, or every
// head in full mode), compacted fixed store if selected, host mirror (+ slot if resident) for tidal heads.
__global__ void __launch_bounds__(128) wnw_place_gather_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                               int full_mode, const bf16 *stage) {
  const Geometry &G = cv.geo;
  const int c = blockIdx.x, h = blockIdx.y;
  const LayerInfo li = cv.layers[layer];
  const long long bl = (long long)b * G.L + layer;
  const int role = full_mode ? ROLE_ANCHOR : cv.roles[layer * G.Hkv + h];
  const int ridx = full_mode ? h : cv.role_idx[layer * G.Hkv + h];
  const int vec_per_chunk = G.ncp * G.d / 8;
  bf16 *dst0[2] = {nullptr, nullptr}, *dst1[2] = {nullptr, nullptr};
  if (role == ROLE_ANCHOR) {
    const int head = full_mode ? layer * G.Hkv + h : li.anchor_off + ridx;
    for (int kv = 0; kv < 2; ++kv) dst0[kv] = cv.anchor + anchor_off(G, G.anchor_seq_stride, b, head, kv) + (long long)c * G.ncp * G.d;
  } else if (role == ROLE_FIXED) {
    const long long fh = (long long)b * G.F_tot + li.fixed_off + ridx;
    int pos = -1;
    for (int s = 0; s < cv.fixed_n[fh]; ++s)
      if (cv.fixed_chunks[fh * G.FB + s] == c) pos = s;
    if (pos < 0) return;
    for (int kv = 0; kv < 2; ++kv) dst0[kv] = cv.fixed + fixed_off(G, li, b, ridx, kv) + (long long)pos * G.ncp * G.d;
  } else if (G.kv8) {
    // e4m3 tidal tier: the staged rows already hold values on the e4m3 grid of the chunk's scale (wnw_quantise_stage_kernel),
    // so the conversion is exact; bytes go out in the order the decode kernel's ldmatrix wants (e4m3_store_pos)
    const int slot = cv.chunk_slot[bl * G.C_max + c];
    const int groups = G.ncp * G.d / 16;
    for (int kv = 0; kv < 2; ++kv) {
      const float inv = exp2f(-(float)cv.kv_exp[kv_exp_off(G, cv.tid_total, b, li.tid_prefix + ridx, c) + kv]);
      const bf16 *src = stage + anchor_off(G, 0, 0, h, kv) + (long long)c * G.ncp * G.d;
      uint4 *m = reinterpret_cast<uint4 *>(tier_ptr(G, cv.mirror[b], mirror_off(G, li, mirror_chunks_of(G, cv.C[b]), c, ridx, kv)));
      uint4 *p = slot >= 0 ? reinterpret_cast<uint4 *>(tier_ptr(G, cv.pool, pool_off(G, li, b, slot, ridx, kv))) : nullptr;
      for (int gidx = threadIdx.x; gidx < groups; gidx += blockDim.x) {
        union { uint4 v; uint8_t b[16]; } out;
#pragma unroll
        for (int e = 0; e < 16; ++e)
          out.b[e4m3_store_pos(kv, e)] =
              (uint8_t)__nv_cvt_float_to_fp8(__bfloat162float(src[(long long)gidx * 16 + e]) * inv, __NV_SATFINITE, __NV_E4M3);
        m[gidx] = out.v;
        if (p) p[gidx] = out.v;
      }
    }
    return;
  } else {
    const int slot = cv.chunk_slot[bl * G.C_max + c];
    for (int kv = 0; kv < 2; ++kv) {
      dst0[kv] = cv.mirror[b] + mirror_off(G, li, mirror_chunks_of(G, cv.C[b]), c, ridx, kv);
      if (slot >= 0) dst1[kv] = cv.pool + pool_off(G, li, b, slot, ridx, kv);
    }
  }
  for (int kv = 0; kv < 2; ++kv) {
    const uint4 *src = reinterpret_cast<const uint4 *>(stage + anchor_off(G, 0, 0, h, kv) + (long long)c * G.ncp * G.d);
    uint4 *d0 = reinterpret_cast<uint4 *>(dst0[kv]), *d1 = reinterpret_cast<uint4 *>(dst1[kv]);
    for (int v = threadIdx.x; v < vec_per_chunk; v += blockDim.x) {
      const uint4 val = src[v];  // staging pad rows are zero
      d0[v] = val;
      if (d1) d1[v] = val;
    }
  }
}
// e4m3 tidal tier, grid (C_b, Hkv), CTAs of tidal heads only.  Per K and V of one chunk of one head: the largest magnitude of
// the staged rows gives the scale exponent e (the integer with max / 2^e in (224, 448], e4m3's top binade; 0 for an all-zero
// block), and every staged element is replaced by e4m3(x / 2^e) * 2^e, rounded to nearest even: the value its byte will
// decode to, an exact bf16 number.
__global__ void __launch_bounds__(128) wnw_quantise_stage_kernel(const __grid_constant__ CacheView cv, int b, int layer, bf16 *stage) {
  const Geometry &G = cv.geo;
  const int c = blockIdx.x, h = blockIdx.y;
  if (cv.roles[layer * G.Hkv + h] != ROLE_TIDAL) return;
  const LayerInfo li = cv.layers[layer];
  const int ridx = cv.role_idx[layer * G.Hkv + h], n = G.ncp * G.d;
  __shared__ unsigned int s_max[4];
  for (int kv = 0; kv < 2; ++kv) {
    bf16 *rows = stage + anchor_off(G, 0, 0, h, kv) + (long long)c * G.ncp * G.d;
    unsigned int mx = 0;   // magnitudes of finite bf16 numbers order like their bit patterns
    for (int i = threadIdx.x; i < n; i += blockDim.x) mx = max(mx, (unsigned int)(__bfloat16_as_ushort(rows[i]) & 0x7fffu));
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = max(max(s_max[0], s_max[1]), max(s_max[2], s_max[3]));
    __syncthreads();
    int e = 0;
    if (mx) {   // max = 1.m * 2^x; 448 = 1.75 * 2^8
      e = (int)(mx >> 7) - 127 - 8 + ((mx & 0x7fu) > 96u ? 1 : 0);
      e = e < -127 ? -127 : (e > 127 ? 127 : e);
    }
    if (threadIdx.x == 0) cv.kv_exp[kv_exp_off(G, cv.tid_total, b, li.tid_prefix + ridx, c) + kv] = (int8_t)e;
    const float inv = exp2f(-(float)e), sc = exp2f((float)e);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const __nv_fp8_storage_t q = __nv_cvt_float_to_fp8(__bfloat162float(rows[i]) * inv, __NV_SATFINITE, __NV_E4M3);
      rows[i] = __float2bfloat16_rn(__half2float(__half(__nv_cvt_fp8_to_halfraw(q, __NV_E4M3))) * sc);
    }
  }
}
cudaError_t launch_quantise_stage(const CacheView &cv, int b, int layer, bf16 *stage, int C_b, cudaStream_t st) {
  if (C_b <= 0 || cv.layers == nullptr) return cudaSuccess;
  wnw_quantise_stage_kernel<<<dim3(C_b, cv.geo.Hkv), 128, 0, st>>>(cv, b, layer, stage);
  return cudaGetLastError();
}

cudaError_t launch_place_gather(const CacheView &cv, int b, int layer, int full_mode, const bf16 *stage, int C_b,
                                  cudaStream_t st) {
  if (C_b <= 0) return cudaSuccess;
  wnw_place_gather_kernel<<<dim3(C_b, cv.geo.Hkv), 128, 0, st>>>(cv, b, layer, full_mode, stage);
  return cudaGetLastError();
}

}  // namespace wnw
