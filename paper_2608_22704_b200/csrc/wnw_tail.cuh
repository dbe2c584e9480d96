// Device-side pieces of the selection: ranking key, top-k, residency update (hard budget; segment lag) and recall plan.
// Included by the selection kernel and the placement kernels (wnw_kernels.cu).
//
// The selection kernel runs one CTA per sequence on a side stream, off the attention's critical path; its cost is pure
// latency.  Everything it reads from global memory is therefore staged into shared memory by cp.async in ONE batch (one
// round trip), and all arithmetic then runs out of shared memory in a fixed order (deterministic scores and selections).
#pragma once
#include "wnw_internal.cuh"

namespace wnw {

__device__ __forceinline__ int chunk_len(const Geometry &G, int T_a, int c) {
  int len = T_a - c * G.nc;
  return len > G.nc ? G.nc : len;
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
    v = w > v ? w : v;
  }
  return v;
}
__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
    v = w < v ? w : v;
  }
  return v;
}

// Ranking key of "Dynamic Chunk Selection": the chunk MEAN as fp32 (IEEE division), ties to the lower chunk
// index.  Scores are >= 0, so the float's bit pattern orders like the value.
__device__ __forceinline__ unsigned long long rank_key(float score_sum, int len, int c) {
  const float key = __fdiv_rn(score_sum, (float)len);
  return ((unsigned long long)__float_as_uint(key) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)c);
}

__device__ __forceinline__ void cp_async_small(void *smem_dst, const void *src, int bytes /* 4, 8 or 16 */) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  if (bytes == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(src) : "memory");
  else if (bytes == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(src) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait_all() {
  asm volatile("cp.async.commit_group;\n" ::: "memory");
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

// Per-warp shared-memory workspace of one table update.
struct SelectWs {
  unsigned long long *keys;  // [C]
  long long *stamp;          // [S]
  int *slot;                 // [S]
  float *sc;                 // [C] scores of a source layer other than the one just computed
};
__device__ __forceinline__ SelectWs select_ws_at(unsigned char *p, int C, int S) {
  SelectWs w;
  w.keys = reinterpret_cast<unsigned long long *>(p);
  w.stamp = reinterpret_cast<long long *>(p + (size_t)C * 8);
  w.slot = reinterpret_cast<int *>(p + (size_t)C * 8 + (size_t)S * 8);
  w.sc = reinterpret_cast<float *>(p + (size_t)C * 8 + (size_t)S * 12);
  return w;
}

// Stage 1 of a table update (one warp): queue the copies of the layer's table and, if needed, of its source
// layer's scores.  The caller commits, waits and synchronises.
__device__ __forceinline__ void select_stage(const CacheView &cv, int b, int lt, int src, bool src_is_local, int C_b, int S_b,
                                             int lane, const SelectWs &w, int parity) {
  const Geometry &G = cv.geo;
  const long long bl = (long long)b * G.L + lt;
  for (int s = lane; s < S_b; s += 32) {
    cp_async_small(w.slot + s, cv.slot_chunk + slot_table_off(G, parity, bl) + s, 4);
    cp_async_small(w.stamp + s, cv.stamp + bl * G.S_max + s, 8);
  }
  if (!src_is_local && src >= 0) {
    const float *sc = cv.score_sum + ((long long)b * G.L + src) * G.C_max;
    for (int c = lane; c < C_b; c += 32) cp_async_small(w.sc + c, sc + c, 4);
  }
}

// Stage 2 (one warp): top-k of layer `lt` from scores `sc` (shared memory), then the residency update (hit:
// refresh stamp; miss: lowest free slot, else least recently selected resident not selected now) and the recall
// plan.  Works on the staged table; global memory only receives stores.
// Returns the number of planned copies (uniform over the warp).
__device__ __forceinline__ int select_and_update(const CacheView &cv, int b, int lt, int src, int C_b, int S_b, int T_a,
                                                  long long step, int lane, const float *sc, const SelectWs &w, int parity) {
  const Geometry &G = cv.geo;
  const long long bl = (long long)b * G.L + lt;
  int k = G.topk < S_b ? G.topk : S_b;
  if (src == -1 || C_b <= 0) k = 0;   // -1: nothing to rank by; -2: the global accumulator
  int *slot_next = cv.slot_chunk + slot_table_off(G, parity ^ 1, bl);   // the whole updated table goes to the other copy
  int *chunk_slot = cv.chunk_slot + bl * G.C_max;
  long long *stamp = cv.stamp + bl * G.S_max;
  if (k > 0)
    for (int c = lane; c < C_b; c += 32) w.keys[c] = rank_key(sc[c], chunk_len(G, T_a, c), c);
  __syncwarp();
  int sel[MAX_TOPK];
  unsigned long long prev = ~0ull;
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0ull;
    for (int c = lane; c < C_b; c += 32) {
      const unsigned long long key = w.keys[c];
      if (key < prev && key > best) best = key;
    }
    best = warp_max_u64(best);
    sel[r] = (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull));
    prev = best;
  }
  int *plan = cv.plan + bl * G.plan_cap * 2;
  int n_plan = 0, hits = 0, evictions = 0;
  for (int r = 0; r < k; ++r) {
    const int c = sel[r];
    const long long st = step * G.topk + (G.topk - 1 - r);
    int j = -1, free_j = 0x7fffffff;
    for (int s = lane; s < S_b; s += 32) {
      const int rc = w.slot[s];
      if (rc == c) j = s;
      if (rc < 0 && s < free_j) free_j = s;
    }
    const unsigned hit_mask = __ballot_sync(0xffffffffu, j >= 0);
    if (hit_mask) {  // hit: refresh recency
      j = __shfl_sync(0xffffffffu, j, __ffs(hit_mask) - 1);
      if (lane == 0) { w.stamp[j] = st; stamp[j] = st; }
      ++hits;
      __syncwarp();
      continue;
    }
    free_j = __reduce_min_sync(0xffffffffu, free_j);
    if (free_j != 0x7fffffff) {
      j = free_j;  // lowest-index free slot
    } else {       // victim: smallest stamp among residents that are not selected now (stamps are unique)
      unsigned long long mykey = ~0ull;
      int myslot = -1;
      for (int s = lane; s < S_b; s += 32) {
        const int rc = w.slot[s];
        bool in_sel = false;
        for (int q = 0; q < k; ++q) in_sel |= sel[q] == rc;
        if (in_sel) continue;
        const unsigned long long key = (unsigned long long)(w.stamp[s] + (1ll << 62));  // order-preserving bias
        if (key < mykey) { mykey = key; myslot = s; }
      }
      const unsigned long long best = warp_min_u64(mykey);
      if (best == ~0ull) {
        if (lane == 0) atomicOr(cv.status, STATUS_NO_VICTIM);
        break;
      }
      const unsigned owner = __ballot_sync(0xffffffffu, mykey == best);
      j = __shfl_sync(0xffffffffu, myslot, __ffs(owner) - 1);
    }
    if (lane == 0) {
      const int old = w.slot[j];
      if (old >= 0) { chunk_slot[old] = -1; ++evictions; }
      w.slot[j] = c; w.stamp[j] = st;
      chunk_slot[c] = j; stamp[j] = st;
      plan[2 * n_plan] = c;
      plan[2 * n_plan + 1] = j;
    }
    ++n_plan;
    __syncwarp();
  }
  __syncwarp();
  for (int s = lane; s < S_b; s += 32) slot_next[s] = w.slot[s];
  if (lane == 0) {
    for (int r = 0; r < k; ++r) cv.sel[bl * G.topk + r] = sel[r];
    cv.n_sel[bl] = k;
    cv.n_plan[bl] = n_plan;
    if (k > 0) {
      atomicAdd(cv.stats + (long long)b * 4 + 0, (unsigned long long)hits);
      atomicAdd(cv.stats + (long long)b * 4 + 1, (unsigned long long)n_plan);
      atomicAdd(cv.stats + (long long)b * 4 + 2, (unsigned long long)evictions);
    }
  }
  return n_plan;
}

// SEGMENT_LAG residency (one warp): chunk j = segments j, j+1 ranked by the mean over its tokens; the segments of the k
// best chunks, in rank order without repeats, are this step's selection.  Slots [0, S_base) never change.  A selected
// segment that is resident is a hit (a dynamic one gets stamp = step); then every dynamic slot not selected now with
// step - stamp >= delta is released; then the misses take the lowest free dynamic slots in order and are planned.
// Returns the number of planned copies (uniform over the warp).
__device__ __forceinline__ int select_and_update_lag(const CacheView &cv, int b, int lt, int src, int C_b, int S_b, int S_base,
                                                      int T_a, long long step, int lane, const float *sc, const SelectWs &w,
                                                      int parity) {
  const Geometry &G = cv.geo;
  const long long bl = (long long)b * G.L + lt;
  const int n_ch = C_b > 1 ? C_b - 1 : C_b;
  int k = G.topk < n_ch ? G.topk : n_ch;
  if (src == -1 || C_b <= 0) k = 0;
  int *slot_next = cv.slot_chunk + slot_table_off(G, parity ^ 1, bl);   // the whole updated table goes to the other copy
  int *chunk_slot = cv.chunk_slot + bl * G.C_max;
  long long *stamp = cv.stamp + bl * G.S_max;
  if (k > 0)
    for (int j = lane; j < n_ch; j += 32) {
      const float sum = C_b > 1 ? __fadd_rn(sc[j], sc[j + 1]) : sc[j];
      const int len = chunk_len(G, T_a, j) + (C_b > 1 ? chunk_len(G, T_a, j + 1) : 0);
      w.keys[j] = rank_key(sum, len, j);
    }
  __syncwarp();
  int sel[MAX_TOPK];
  unsigned long long prev = ~0ull;
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0ull;
    for (int j = lane; j < n_ch; j += 32) {
      const unsigned long long key = w.keys[j];
      if (key < prev && key > best) best = key;
    }
    best = warp_max_u64(best);
    sel[r] = (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull));
    prev = best;
  }
  int segs[2 * MAX_TOPK];
  int n_seg = 0;
  for (int r = 0; r < k; ++r)
    for (int e = 0; e < (C_b > 1 ? 2 : 1); ++e) {
      const int g = sel[r] + e;
      bool seen = false;
      for (int i = 0; i < n_seg; ++i) seen |= segs[i] == g;
      if (!seen) segs[n_seg++] = g;
    }
  // hits
  unsigned miss = 0;
  int hits = 0;
  for (int i = 0; i < n_seg; ++i) {
    int j = -1;
    for (int s = lane; s < S_b; s += 32)
      if (w.slot[s] == segs[i]) j = s;
    const unsigned hit_mask = __ballot_sync(0xffffffffu, j >= 0);
    if (!hit_mask) { miss |= 1u << i; continue; }
    j = __shfl_sync(0xffffffffu, j, __ffs(hit_mask) - 1);
    ++hits;
    if (j >= S_base && lane == 0) { w.stamp[j] = step; stamp[j] = step; }
  }
  __syncwarp();
  // release what has gone unselected for delta steps
  int released = 0;
  for (int s0 = S_base; s0 < S_b; s0 += 32) {
    const int s = s0 + lane;
    bool drop = false;
    if (s < S_b) {
      const int rc = w.slot[s];
      drop = rc >= 0 && w.stamp[s] != step && step - w.stamp[s] >= (long long)G.delta;
      if (drop) { w.slot[s] = -1; chunk_slot[rc] = -1; }
    }
    released += __popc(__ballot_sync(0xffffffffu, drop));
  }
  __syncwarp();
  // misses, in order, into the lowest free dynamic slots
  int *plan = cv.plan + bl * G.plan_cap * 2;
  int n_plan = 0;
  for (int i = 0; i < n_seg; ++i) {
    if (!(miss >> i & 1u)) continue;
    int free_j = 0x7fffffff;
    for (int s = S_base + lane; s < S_b; s += 32)
      if (w.slot[s] < 0 && s < free_j) free_j = s;
    free_j = __reduce_min_sync(0xffffffffu, free_j);
    if (free_j == 0x7fffffff) {   // cannot happen: 2k(delta+1) dynamic slots always suffice
      if (lane == 0) atomicOr(cv.status, STATUS_NO_VICTIM);
      break;
    }
    if (lane == 0) {
      w.slot[free_j] = segs[i]; w.stamp[free_j] = step;
      chunk_slot[segs[i]] = free_j; stamp[free_j] = step;
      plan[2 * n_plan] = segs[i];
      plan[2 * n_plan + 1] = free_j;
    }
    ++n_plan;
    __syncwarp();
  }
  __syncwarp();
  for (int s = lane; s < S_b; s += 32) slot_next[s] = w.slot[s];
  if (lane == 0) {
    for (int r = 0; r < k; ++r) cv.sel[bl * G.topk + r] = sel[r];
    cv.n_sel[bl] = k;
    cv.n_plan[bl] = n_plan;
    if (k > 0) {
      atomicAdd(cv.stats + (long long)b * 4 + 0, (unsigned long long)hits);
      atomicAdd(cv.stats + (long long)b * 4 + 1, (unsigned long long)n_plan);
      atomicAdd(cv.stats + (long long)b * 4 + 2, (unsigned long long)released);
    }
  }
  return n_plan;
}

}  // namespace wnw
