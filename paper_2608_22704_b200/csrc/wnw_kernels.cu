// Tail (split merge, chunk-score finalize, top-k, residency update, recall plan), recall, text append,
// step bookkeeping and prefill placement kernels (sm_100a).
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

// One warp: top-k of layer `lt` of sequence b from the scores of its source layer, then the residency update
// (hit: refresh stamp; miss: lowest free slot, else least recently selected resident not selected now) and the
// recall plan.  The new table is read by attention from the next step on.
__device__ void select_and_update(const CacheView &cv, int b, int lt, int lane) {
  const Geometry &G = cv.geo;
  const LayerInfo li = cv.layers[lt];
  const int C_b = cv.C[b], S_b = cv.S[b], T_a = cv.T_a[b];
  const long long bl = (long long)b * G.L + lt;
  int k = G.topk < S_b ? G.topk : S_b;
  if (li.src < 0 || C_b <= 0) k = 0;
  int sel[MAX_TOPK];
  const float *sc = cv.score_sum + ((long long)b * G.L + li.src) * G.C_max;
  unsigned long long prev = ~0ull;
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0ull;
    for (int c = lane; c < C_b; c += 32) {
      const float s = __ldcg(sc + c);
      const unsigned long long key = rank_key(s, chunk_len(G, T_a, c), c);
      if (key < prev && key > best) best = key;
    }
    best = warp_max_u64(best);
    sel[r] = (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull));
    prev = best;
  }
  int *slot_chunk = cv.slot_chunk + bl * G.S_max;
  int *chunk_slot = cv.chunk_slot + bl * G.C_max;
  long long *stamp = cv.stamp + bl * G.S_max;
  int *plan = cv.plan + bl * G.topk * 2;
  const long long step = cv.steps[b];
  int n_plan = 0, hits = 0, evictions = 0;
  for (int r = 0; r < k; ++r) {
    const int c = sel[r];
    const long long st = step * G.topk + (G.topk - 1 - r);
    int j = chunk_slot[c];
    if (j >= 0) {
      if (lane == 0) stamp[j] = st;
      ++hits;
      __syncwarp();
      continue;
    }
    // lowest-index free slot
    unsigned long long cand = ~0ull;
    for (int s = lane; s < S_b; s += 32)
      if (slot_chunk[s] < 0) { cand = (unsigned long long)s; break; }
    cand = warp_min_u64(cand);
    if (cand != ~0ull) {
      j = (int)cand;
    } else {  // victim: smallest stamp among residents that are not selected now (stamps are unique)
      unsigned long long mykey = ~0ull;
      int myslot = -1;
      for (int s = lane; s < S_b; s += 32) {
        const int rc = slot_chunk[s];
        bool in_sel = false;
        for (int q = 0; q < k; ++q) in_sel |= sel[q] == rc;
        if (in_sel) continue;
        const unsigned long long key = (unsigned long long)(stamp[s] + (1ll << 62));  // order-preserving bias
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
    __syncwarp();
    if (lane == 0) {
      const int old = slot_chunk[j];
      if (old >= 0) { chunk_slot[old] = -1; ++evictions; }
      slot_chunk[j] = c;
      chunk_slot[c] = j;
      stamp[j] = st;
      plan[2 * n_plan] = c;
      plan[2 * n_plan + 1] = j;
    }
    ++n_plan;
    __syncwarp();
  }
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
}

// grid (Hkv, n_active).  Merges the split partials of one (sequence, KV head) into bf16 outputs; the CTA that
// finishes a sequence last finalizes this layer's chunk scores and runs selection for every layer whose score
// source is now complete.
__global__ void __launch_bounds__(256) wnw_tail_kernel(const __grid_constant__ CacheView cv,
                                                       const __grid_constant__ TailArgs a) {
  extern __shared__ float sm_w[];  // [count][g] weights, then [count][g] l
  __shared__ float sM[MAX_G], sZ[MAX_G];
  __shared__ int s_last;
  const Geometry &G = cv.geo;
  const int h = blockIdx.x, i = blockIdx.y, b = a.active[i];
  const int g = G.g, D = G.d, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const HeadItems hi = a.head_items[i * G.Hkv + h];
  float *sm_l = sm_w + hi.count * g;
  for (int idx = tid; idx < hi.count * g; idx += blockDim.x) {
    const float2 ml = __ldcg(a.part_ml + (long long)hi.first * g + idx);
    sm_w[idx] = ml.x;
    sm_l[idx] = ml.y;
  }
  __syncthreads();
  for (int row = warp; row < g; row += 8) {
    float M = -INFINITY;
    for (int n = lane; n < hi.count; n += 32) M = fmaxf(M, sm_w[n * g + row]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float Z = 0.f;
    for (int n = lane; n < hi.count; n += 32) {
      const float w = M > -INFINITY ? exp2f(sm_w[n * g + row] - M) : 0.f;
      sm_w[n * g + row] = w;
      Z += sm_l[n * g + row] * w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
    if (lane == 0) {
      sM[row] = M; sZ[row] = Z;
      a.head_mz[(long long)i * G.Hq + h * g + row] = make_float2(M, Z);
    }
  }
  __syncthreads();
  if (a.out != nullptr) {
    for (int idx = tid; idx < g * D; idx += blockDim.x) {
      const int row = idx / D, col = idx - row * D;
      float acc = 0.f;
      const float *po = a.part_o + ((long long)hi.first * g + row) * D + col;
      for (int n = 0; n < hi.count; ++n) acc += __ldcg(po + (long long)n * g * D) * sm_w[n * g + row];
      const float Z = sZ[row];
      a.out[((long long)i * G.Hq + h * g + row) * D + col] = __float2bfloat16_rn(Z > 0.f ? acc / Z : 0.f);
    }
  }
  if (a.mode != ATTN_DECODE) return;

  // ---- last CTA of this sequence: scores, selection, table update ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(a.seq_done + i, 1);
    s_last = prev == G.Hkv - 1;
    if (s_last) a.seq_done[i] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const LayerInfo li = cv.layers[a.layer];
  const int C_b = cv.C[b], T_a = cv.T_a[b];
  if (li.n_anchor > 0 && a.score_on) {
    float *dst = cv.score_sum + ((long long)b * G.L + a.layer) * G.C_max;
    for (int c = tid; c < C_b; c += blockDim.x) {
      float total = 0.f;
      int aidx = 0;
      for (int hh = 0; hh < G.Hkv; ++hh) {
        if (cv.roles[a.layer * G.Hkv + hh] != ROLE_ANCHOR) continue;
        for (int r = 0; r < g; ++r) {
          const float2 mz = __ldcg(a.head_mz + (long long)i * G.Hq + hh * g + r);
          const float2 *ge = a.gran_em + ((long long)i * a.n_aq + (long long)aidx * g + r) * a.n_ag_max + (long long)c * G.gpc;
          float sum_h = 0.f;
          for (int gi = 0; gi < G.gpc; ++gi) {
            if (c * G.nc + gi * GR >= T_a) break;
            const float2 em = __ldcg(ge + gi);
            sum_h += em.x * exp2f(em.y - mz.x);
          }
          total += mz.y > 0.f ? sum_h / mz.y : 0.f;
        }
        ++aidx;
      }
      if (!(total >= 0.f) || isinf(total)) atomicOr(cv.status, STATUS_NONFINITE);
      dst[c] = total;
    }
  }
  __syncthreads();
  for (int u = warp; u < li.upd_count; u += 8) select_and_update(cv, b, cv.upd_list[li.upd_first + u], lane);
}

// max_count: the largest number of work items of any (sequence, KV head) in this launch (sizes shared memory).
cudaError_t launch_tail(const CacheView &cv, const TailArgs &a, int max_count, cudaStream_t st) {
  const size_t smem = (size_t)max_count * cv.geo.g * 2 * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  if (smem > 48 * 1024) {
    static size_t configured = 0;
    if (smem > configured) {
      cudaError_t e = cudaFuncSetAttribute(wnw_tail_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      configured = smem;
    }
  }
  wnw_tail_kernel<<<dim3(cv.geo.Hkv, a.n_active), 256, smem, st>>>(cv, a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Recall: copies every planned chunk block pinned host -> slot pool.  grid (ctas, topk, n_active * n_layers).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) wnw_recall_kernel(const __grid_constant__ CacheView cv, int n_active,
                                                         const int32_t *active, const int32_t *layers, int n_layers,
                                                         int skip_copy) {
  const Geometry &G = cv.geo;
  const int i = blockIdx.z / n_layers, l = layers[blockIdx.z % n_layers], r = blockIdx.y;
  const int b = active[i];
  const long long bl = (long long)b * G.L + l;
  if (r >= cv.n_plan[bl]) return;
  const LayerInfo li = cv.layers[l];
  const int c = cv.plan[(bl * G.topk + r) * 2], slot = cv.plan[(bl * G.topk + r) * 2 + 1];
  const long long n_vec = (long long)li.n_tidal * 2 * G.nc * G.d / 8;  // 16-byte vectors per chunk block
  if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(cv.stats + (long long)b * 4 + 3, (unsigned long long)n_vec * 16ull);
  if (skip_copy) return;
  if (c < 0 || c >= cv.C[b] || slot < 0 || slot >= cv.S[b]) {
    if (threadIdx.x == 0) atomicOr(cv.status, STATUS_BAD_TABLE);
    return;
  }
  const uint4 *src = reinterpret_cast<const uint4 *>(cv.mirror[b] + mirror_off(G, li, cv.C[b], c, 0, 0));
  uint4 *dst = reinterpret_cast<uint4 *>(cv.pool + pool_off(G, li, b, slot, 0, 0));
  constexpr int U = 8;
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

cudaError_t launch_recall(const CacheView &cv, int n_active, const int32_t *active, const int32_t *layers_dev, int n_layers,
                          int skip_copy, cudaStream_t st) {
  if (n_layers <= 0 || n_active <= 0) return cudaSuccess;
  wnw_recall_kernel<<<dim3(8, cv.geo.topk, n_active * n_layers), 256, 0, st>>>(cv, n_active, active, layers_dev, n_layers,
                                                                            skip_copy);
  return cudaGetLastError();
}

// Plain host-mapped -> device copy with the recall kernel's access pattern (link probe).
__global__ void __launch_bounds__(256) wnw_copy_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, long long n_vec) {
  constexpr int U = 8;
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
// Text append and step bookkeeping
// ------------------------------------------------------------------------------------------------
__global__ void wnw_append_kernel(const __grid_constant__ CacheView cv, int layer, const int32_t *active, const bf16 *k_new,
                                  const bf16 *v_new) {
  const Geometry &G = cv.geo;
  const int i = blockIdx.x, b = active[i];
  const int row = cv.text_len[b];
  if (row >= G.T_cap_pad) {
    if (threadIdx.x == 0) atomicOr(cv.status, STATUS_BAD_TABLE);
    return;
  }
  const int vec_per_head = G.d / 8;
  for (int idx = threadIdx.x; idx < G.Hkv * vec_per_head * 2; idx += blockDim.x) {
    const int kv = idx / (G.Hkv * vec_per_head), rem = idx - kv * G.Hkv * vec_per_head;
    const int h = rem / vec_per_head, v = rem - h * vec_per_head;
    const bf16 *src = (kv ? v_new : k_new) + ((long long)i * G.Hkv + h) * G.d + v * 8;
    bf16 *dst = cv.text + text_off(G, b, layer, h, kv) + (long long)row * G.d + v * 8;
    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
  }
}
cudaError_t launch_append(const CacheView &cv, int layer, int n_active, const int32_t *active, const bf16 *k_new,
                          const bf16 *v_new, cudaStream_t st) {
  wnw_append_kernel<<<n_active, 128, 0, st>>>(cv, layer, active, k_new, v_new);
  return cudaGetLastError();
}

__global__ void wnw_step_end_kernel(const __grid_constant__ CacheView cv, int n_active, const int32_t *active, int appended) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_active) return;
  const int b = active[i];
  cv.steps[b] += 1;
  if (appended) cv.text_len[b] += 1;
}
cudaError_t launch_step_end(const CacheView &cv, int n_active, const int32_t *active, int appended, cudaStream_t st) {
  wnw_step_end_kernel<<<(n_active + 127) / 128, 128, 0, st>>>(cv, n_active, active, appended);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Prefill placement ("Prefill Compression", chunk level)
// ------------------------------------------------------------------------------------------------

// Splits one layer's prefill K,V [n_tokens][Hkv][d] into the text store and a per-head staging copy of the audio
// (anchor layout [Hkv][K|V][T_a_pad][d]), zero-pads the staging tail, and resets the layer's tables.
__global__ void __launch_bounds__(256) wnw_place_scatter_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                const bf16 *k, const bf16 *v, int n_tokens, int ab, int ae,
                                                                int T_t, int C_b, int S_b, bf16 *stage) {
  const Geometry &G = cv.geo;
  const int T_a = ae - ab, vec_per_row = G.d / 8;
  const long long bl = (long long)b * G.L + layer;
  if (blockIdx.x == 0) {
    if (threadIdx.x == 0) {
      cv.text_len[b] = T_t; cv.T_a[b] = T_a; cv.C[b] = C_b; cv.S[b] = S_b;
      cv.n_sel[bl] = 0; cv.n_plan[bl] = 0;
      if (layer == 0) {
        cv.steps[b] = 0;
        for (int x = 0; x < 4; ++x) cv.stats[(long long)b * 4 + x] = 0ull;
      }
    }
    for (int s = threadIdx.x; s < G.S_max; s += blockDim.x) { cv.slot_chunk[bl * G.S_max + s] = -1; cv.stamp[bl * G.S_max + s] = 0; }
    for (int c = threadIdx.x; c < G.C_max; c += blockDim.x) { cv.chunk_slot[bl * G.C_max + c] = -1; cv.score_sum[bl * G.C_max + c] = 0.f; }
    const LayerInfo li = cv.layers[layer];
    for (int f = threadIdx.x; f < li.n_fixed; f += blockDim.x) cv.fixed_n[(long long)b * G.F_tot + li.fixed_off + f] = 0;
  }
  const int rows_total = n_tokens + (C_b * G.nc - T_a);  // real tokens, then staging pad rows
  const long long work = (long long)rows_total * G.Hkv * 2 * vec_per_row;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < work; idx += (long long)gridDim.x * blockDim.x) {
    const int vv = (int)(idx % vec_per_row);
    long long t = idx / vec_per_row;
    const int kv = (int)(t % 2); t /= 2;
    const int h = (int)(t % G.Hkv);
    const int tok = (int)(t / G.Hkv);
    uint4 val = make_uint4(0, 0, 0, 0);
    bf16 *dst;
    if (tok < n_tokens) {
      val = *reinterpret_cast<const uint4 *>((kv ? v : k) + ((long long)tok * G.Hkv + h) * G.d + vv * 8);
      if (tok >= ab && tok < ae) dst = stage + anchor_off(G, 0, 0, h, kv) + (long long)(tok - ab) * G.d + vv * 8;
      else dst = cv.text + text_off(G, b, layer, h, kv) + (long long)(tok < ab ? tok : tok - T_a) * G.d + vv * 8;
    } else {
      dst = stage + anchor_off(G, 0, 0, h, kv) + (long long)(T_a + (tok - n_tokens)) * G.d + vv * 8;
    }
    *reinterpret_cast<uint4 *>(dst) = val;
  }
}
cudaError_t launch_place_scatter(const CacheView &cv, int b, int layer, const bf16 *k, const bf16 *v, int n_tokens, int ab,
                                 int ae, int T_t, int C_b, int S_b, bf16 *stage, cudaStream_t st) {
  wnw_place_scatter_kernel<<<296, 256, 0, st>>>(cv, b, layer, k, v, n_tokens, ab, ae, T_t, C_b, S_b, stage);
  return cudaGetLastError();
}

// One CTA.  From the prefill attention partials of q_last: pre[h][c] per non-anchor KV head, then the fixed heads'
// own top-S sets and the tidal heads' shared top-S table (rank r -> slot r, stamp -1-r).
__global__ void __launch_bounds__(512) wnw_prefill_select_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                 const HeadItems *head_items, const float2 *part_ml,
                                                                 const float2 *gran_em, int n_ag_max) {
  extern __shared__ float sm[];  // [Hq] M, [Hq] Z, [C_max] keys (as u64 pairs)
  const Geometry &G = cv.geo;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarp = blockDim.x >> 5;
  const int g = G.g, C_b = cv.C[b], S_b = cv.S[b], T_a = cv.T_a[b];
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
          if (c * G.nc + gi * GR >= T_a) break;
          sum_h += ge[gi].x * exp2f(ge[gi].y - sM[hq]);
        }
        total += sZ[hq] > 0.f ? sum_h / sZ[hq] : 0.f;
      }
    }
    pre[(long long)h * G.C_max + c] = total;
  }
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
      if (rank < S_b) cv.fixed_chunks[fh * G.S_max + rank] = c;
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
        cv.slot_chunk[bl * G.S_max + rank] = c;
        cv.chunk_slot[bl * G.C_max + c] = rank;
        cv.stamp[bl * G.S_max + rank] = -1 - (long long)rank;
      }
    }
  }
}
cudaError_t launch_prefill_select(const CacheView &cv, int b, int layer, const HeadItems *head_items, const float2 *part_ml,
                                  const float2 *gran_em, int n_ag_max, cudaStream_t st) {
  const size_t smem = (size_t)(2 * cv.geo.Hq + 2) * sizeof(float) + (size_t)cv.geo.C_max * sizeof(unsigned long long);
  wnw_prefill_select_kernel<<<1, 512, smem, st>>>(cv, b, layer, head_items, part_ml, gran_em, n_ag_max);
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
  const int vec_per_chunk = G.nc * G.d / 8;
  bf16 *dst0[2] = {nullptr, nullptr}, *dst1[2] = {nullptr, nullptr};
  if (role == ROLE_ANCHOR) {
    const int head = full_mode ? layer * G.Hkv + h : li.anchor_off + ridx;
    for (int kv = 0; kv < 2; ++kv) dst0[kv] = cv.anchor + anchor_off(G, G.anchor_seq_stride, b, head, kv) + (long long)c * G.nc * G.d;
  } else if (role == ROLE_FIXED) {
    const long long fh = (long long)b * G.F_tot + li.fixed_off + ridx;
    int pos = -1;
    for (int s = 0; s < cv.fixed_n[fh]; ++s)
      if (cv.fixed_chunks[fh * G.S_max + s] == c) pos = s;
    if (pos < 0) return;
    for (int kv = 0; kv < 2; ++kv) dst0[kv] = cv.fixed + fixed_off(G, li, b, ridx, kv) + (long long)pos * G.nc * G.d;
  } else {
    const int slot = cv.chunk_slot[bl * G.C_max + c];
    for (int kv = 0; kv < 2; ++kv) {
      dst0[kv] = cv.mirror[b] + mirror_off(G, li, cv.C[b], c, ridx, kv);
      if (slot >= 0) dst1[kv] = cv.pool + pool_off(G, li, b, slot, ridx, kv);
    }
  }
  for (int kv = 0; kv < 2; ++kv) {
    const uint4 *src = reinterpret_cast<const uint4 *>(stage + anchor_off(G, 0, 0, h, kv) + (long long)c * G.nc * G.d);
    uint4 *d0 = reinterpret_cast<uint4 *>(dst0[kv]), *d1 = reinterpret_cast<uint4 *>(dst1[kv]);
    for (int v = threadIdx.x; v < vec_per_chunk; v += blockDim.x) {
      const uint4 val = src[v];  // staging pad rows are zero
      d0[v] = val;
      if (d1) d1[v] = val;
    }
  }
}
cudaError_t launch_place_gather(const CacheView &cv, int b, int layer, int full_mode, const bf16 *stage, int C_b,
                                  cudaStream_t st) {
  if (C_b <= 0) return cudaSuccess;
  wnw_place_gather_kernel<<<dim3(C_b, cv.geo.Hkv), 128, 0, st>>>(cv, b, layer, full_mode, stage);
  return cudaGetLastError();
}

}  // namespace wnw
