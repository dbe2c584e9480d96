// Token-granular prefill compression of fixed heads, and of tidal heads' permanent base ("Prefill Compression";
// retention per head from Eq. 1).
//
// Runs once per (sequence, layer) at placement, after the chunk-granular placement has staged the prefix: the staging
// buffer holds every head's audio K,V in the chunk-padded row layout and the text store holds the text rows.
//   1. wnw_token_score_kernel : p[tau] = sum over the text queries and the head's q-heads of the softmax weight of audio
//                               position tau (softmax over the whole prefix), fp32, one CTA per fixed head, passes in a
//                               fixed order so that the sums are reproducible;
//   2. wnw_token_select_kernel: per segment of n_s tokens the floor(retention * length) positions with the largest p
//                               (equal p: the earlier position), or the same total from the whole head (the ablation's
//                               global top-k); kept positions in ascending order; block table of the compact store;
//   3. wnw_token_gather_kernel: K,V rows of the kept positions from staging into the head's compact fixed store.
// The decode kernel then reads a fixed head as blocks of nc rows whose table entries carry their row count (-(2 + rows))
// instead of a chunk id.
#include "wnw_internal.cuh"

namespace wnw {

namespace {

constexpr int TOK_THREADS = 512;

// Compressed head x of a layer: the fixed heads first, then (token-granular tidal bases) the tidal heads.  Returns the
// KV-head, and in `head` its index among the sequence's compact stores.
__device__ __forceinline__ int comp_head(const CacheView &cv, int layer, int x, int &head) {
  const Geometry &G = cv.geo;
  const LayerInfo &li = cv.layers[layer];
  const int role = x < li.n_fixed ? ROLE_FIXED : ROLE_TIDAL, idx = x < li.n_fixed ? x : x - li.n_fixed;
  head = role == ROLE_FIXED ? li.fixed_off + idx : G.F_fix + li.tid_prefix + idx;
  for (int h = 0; h < G.Hkv; ++h)
    if (cv.roles[layer * G.Hkv + h] == role && cv.role_idx[layer * G.Hkv + h] == idx) return h;
  return -1;
}

__device__ __forceinline__ float block_max(float v, float *red) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float r = red[0];
  for (int i = 1; i < TOK_THREADS / 32; ++i) r = fmaxf(r, red[i]);
  return r;
}
__device__ __forceinline__ float block_sum(float v, float *red) {   // fixed tree: the same bits on every run
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float r = red[0];
  for (int i = 1; i < TOK_THREADS / 32; ++i) r += red[i];
  return r;
}

}  // namespace

// grid: fixed heads of the layer; block: TOK_THREADS.  work: [n_fixed][T_t + T_a] fp32; p_tok: [n_fixed][p_stride] fp32.
__global__ void __launch_bounds__(TOK_THREADS) wnw_token_score_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                     const bf16 *stage, const bf16 *q_text, int n_q, int T_t,
                                                                     int T_a, float *work, float *p_tok, long long p_stride) {
  const Geometry &G = cv.geo;
  extern __shared__ float tok_smem[];
  float *qf = tok_smem, *red = tok_smem + G.d;
  int head;
  const int f = blockIdx.x, h = comp_head(cv, layer, f, head);
  if (h < 0) return;
  const int n = T_t + T_a, d = G.d, pieces = d / 8;
  float *lg = work + (long long)f * (T_t + T_a), *p = p_tok + (long long)f * p_stride;
  const bf16 *tK = cv.text + text_off(G, b, layer, h, 0), *aK = stage + anchor_off(G, 0, 0, h, 0);
  for (int t = threadIdx.x; t < T_a; t += TOK_THREADS) p[t] = 0.f;
  for (int qi = 0; qi < n_q; ++qi)
    for (int j = 0; j < G.g; ++j) {
      __syncthreads();
      const bf16 *q = q_text + ((long long)qi * G.Hq + h * G.g + j) * d;
      for (int x = threadIdx.x; x < d; x += TOK_THREADS) qf[x] = __bfloat162float(q[x]);
      __syncthreads();
      float mx = -INFINITY;
      for (int i = threadIdx.x; i < n; i += TOK_THREADS) {
        const bf16 *row;
        if (i < T_t) row = tK + (long long)i * d;
        else { const int tau = i - T_t; row = aK + ((long long)(tau / G.nc) * G.ncp + tau % G.nc) * d; }
        const uint4 *r4 = reinterpret_cast<const uint4 *>(row);
        float acc = 0.f;
        for (int v = 0; v < pieces; ++v) {
          const uint4 u = r4[v];
          const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 kf = __bfloat1622float2(h2[e]);
            acc = fmaf(qf[v * 8 + 2 * e], kf.x, acc);
            acc = fmaf(qf[v * 8 + 2 * e + 1], kf.y, acc);
          }
        }
        const float l2 = acc * G.scale_log2;
        lg[i] = l2;
        mx = fmaxf(mx, l2);
      }
      mx = block_max(mx, red);
      float z = 0.f;
      for (int i = threadIdx.x; i < n; i += TOK_THREADS) {
        const float e = exp2f(lg[i] - mx);
        lg[i] = e;
        z += e;
      }
      z = block_sum(z, red);
      for (int t = threadIdx.x; t < T_a; t += TOK_THREADS) p[t] += __fdiv_rn(lg[T_t + t], z);
    }
}

// grid: fixed heads of the layer; block: TOK_THREADS.  flags: [n_fixed][p_stride] int32 scratch.
__global__ void __launch_bounds__(TOK_THREADS) wnw_token_select_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                                      const float *p_tok, long long p_stride, int T_a, int seg,
                                                                      const float *retention, int variant, int32_t *flags,
                                                                      int32_t *fixed_tok, int tok_cap, int32_t *tok_n) {
  const Geometry &G = cv.geo;
  __shared__ int counts[TOK_THREADS + 1];
  int head;
  const int f = blockIdx.x, h = comp_head(cv, layer, f, head);
  if (h < 0) return;
  const long long fh = (long long)b * G.F_tot + head;
  const float *key = p_tok + (long long)f * p_stride;
  int32_t *fl = flags + (long long)f * p_stride, *out = fixed_tok + fh * tok_cap;
  const double ret = (double)retention[h];
  int total = 0;
  if (variant != 0)
    for (int lo = 0; lo < T_a; lo += seg) total += (int)floor(ret * (double)min(seg, T_a - lo));
  for (int tau = threadIdx.x; tau < T_a; tau += TOK_THREADS) {
    const float me = key[tau];
    int lo = 0, hi = T_a, m = total;
    if (variant == 0) {
      lo = tau / seg * seg; hi = min(lo + seg, T_a);
      m = (int)floor(ret * (double)(hi - lo));
    }
    int rank = 0;
    for (int t = lo; t < hi && rank < m; ++t) rank += (key[t] > me) || (key[t] == me && t < tau);
    fl[tau] = rank < m;
  }
  __syncthreads();
  // kept positions in ascending order: every thread owns a contiguous range of positions
  const int per = (T_a + TOK_THREADS - 1) / TOK_THREADS, t0 = min(T_a, (int)threadIdx.x * per), t1 = min(T_a, t0 + per);
  int cnt = 0;
  for (int t = t0; t < t1; ++t) cnt += fl[t];
  counts[threadIdx.x] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int i = 0; i < TOK_THREADS; ++i) { const int c = counts[i]; counts[i] = run; run += c; }
    counts[TOK_THREADS] = run;
  }
  __syncthreads();
  int at = counts[threadIdx.x];
  for (int t = t0; t < t1; ++t)
    if (fl[t]) out[at++] = t;
  const int n = counts[TOK_THREADS], n_blk = (n + G.nc - 1) / G.nc;
  for (int s = threadIdx.x; s < G.FB; s += TOK_THREADS)   // block s of the compact store holds min(nc, n - s*nc) rows
    cv.fixed_chunks[fh * G.FB + s] = s < n_blk ? -(2 + min(G.nc, n - s * G.nc)) : -1;
  if (threadIdx.x == 0) { cv.fixed_n[fh] = n_blk; tok_n[fh] = n; }
  const LayerInfo &li = cv.layers[layer];
  if (f >= li.n_fixed) {   // a tidal head's base: how many positions of every segment it holds (what a fetched segment must skip)
    int32_t *sk = cv.seg_kept + ((long long)b * cv.tid_total + li.tid_prefix + (f - li.n_fixed)) * G.C_max;
    for (int c = threadIdx.x; c * G.nc < T_a; c += TOK_THREADS) {
      int k = 0;
      for (int t = c * G.nc; t < min(T_a, (c + 1) * G.nc); ++t) k += fl[t];
      sk[c] = k;
    }
  }
}

// grid (FB, fixed heads of the layer); block 128.  Fills block blockIdx.x of the head's compact store.
__global__ void __launch_bounds__(128) wnw_token_gather_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                               const bf16 *stage, const int32_t *fixed_tok, int tok_cap,
                                                               const int32_t *tok_n) {
  const Geometry &G = cv.geo;
  int head;
  const int blk = blockIdx.x, f = blockIdx.y, h = comp_head(cv, layer, f, head);
  if (h < 0) return;
  const long long fh = (long long)b * G.F_tot + head;
  const int n = tok_n[fh];
  if (blk * G.nc >= n) return;
  const int pieces = G.d / 8;
  const int32_t *pos = fixed_tok + fh * tok_cap;
  for (int kv = 0; kv < 2; ++kv) {
    const uint4 *src = reinterpret_cast<const uint4 *>(stage + anchor_off(G, 0, 0, h, kv));
    uint4 *dst = reinterpret_cast<uint4 *>(cv.fixed + compact_off(G, b, head, kv) + (long long)blk * G.ncp * G.d);
    for (int v = threadIdx.x; v < G.ncp * pieces; v += blockDim.x) {
      const int r = v / pieces, x = v - r * pieces, i = blk * G.nc + r;
      uint4 val = make_uint4(0, 0, 0, 0);   // rows past the block's last token are zero
      if (r < G.nc && i < n) {
        const int tau = pos[i];
        val = src[((long long)(tau / G.nc) * G.ncp + tau % G.nc) * pieces + x];
      }
      dst[v] = val;
    }
  }
}

// grid (segments, tidal heads of the layer); block 128.  Token-granular tidal base: rewrites segment blockIdx.x of the
// head's host mirror with the positions that are NOT in the base first (ascending), the kept ones after them, so that
// the first (length - kept) rows of a fetched segment are exactly its complement.
__global__ void __launch_bounds__(128) wnw_token_mirror_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                               const bf16 *stage, const int32_t *flags, long long p_stride,
                                                               int T_a) {
  const Geometry &G = cv.geo;
  extern __shared__ int mirror_dst[];   // [nc] destination row of every position of the segment
  const LayerInfo li = cv.layers[layer];
  const int c = blockIdx.x, t = blockIdx.y, x = li.n_fixed + t;
  int head;
  const int h = comp_head(cv, layer, x, head);
  if (h < 0) return;
  const int lo = c * G.nc, len = min(G.nc, T_a - lo);
  const int32_t *fl = flags + (long long)x * p_stride + lo;
  int n_out = 0;
  for (int r = 0; r < len; ++r) n_out += fl[r] == 0;
  for (int r = threadIdx.x; r < len; r += blockDim.x) {
    int before_same = 0;
    for (int q = 0; q < r; ++q) before_same += fl[q] == fl[r];
    mirror_dst[r] = fl[r] ? n_out + before_same : before_same;
  }
  __syncthreads();
  const int pieces = G.d / 8;
  for (int kv = 0; kv < 2; ++kv) {
    const uint4 *src = reinterpret_cast<const uint4 *>(stage + anchor_off(G, 0, 0, h, kv) + (long long)c * G.ncp * G.d);
    uint4 *dst = reinterpret_cast<uint4 *>(cv.mirror[b] + mirror_off(G, li, mirror_chunks_of(G, cv.C[b]), c, t, kv));
    for (int v = threadIdx.x; v < len * pieces; v += blockDim.x) {
      const int r = v / pieces, piece = v - r * pieces;
      dst[(long long)mirror_dst[r] * pieces + piece] = src[v];
    }
  }
}

// n_comp: compressed heads of the layer (its fixed heads, then its tidal heads when they keep a token base)
cudaError_t launch_token_compress(const CacheView &cv, int b, int layer, int n_comp, int n_tidal_base, const bf16 *stage,
                                  const bf16 *q_text, int n_q, int T_t, int T_a, int seg, const float *retention_dev,
                                  int variant, float *work, float *p_tok, int32_t *flags, long long p_stride,
                                  int32_t *fixed_tok, int tok_cap, int32_t *tok_n, cudaStream_t st) {
  if (n_comp <= 0 || T_a <= 0) return cudaSuccess;
  const size_t smem = (size_t)(cv.geo.d + TOK_THREADS / 32) * sizeof(float);
  wnw_token_score_kernel<<<n_comp, TOK_THREADS, smem, st>>>(cv, b, layer, stage, q_text, n_q, T_t, T_a, work, p_tok, p_stride);
  wnw_token_select_kernel<<<n_comp, TOK_THREADS, 0, st>>>(cv, b, layer, p_tok, p_stride, T_a, seg, retention_dev, variant, flags,
                                                         fixed_tok, tok_cap, tok_n);
  wnw_token_gather_kernel<<<dim3(cv.geo.FB, n_comp), 128, 0, st>>>(cv, b, layer, stage, fixed_tok, tok_cap, tok_n);
  if (n_tidal_base > 0) {
    const int C_b = (T_a + cv.geo.nc - 1) / cv.geo.nc;
    wnw_token_mirror_kernel<<<dim3(C_b, n_tidal_base), 128, (size_t)cv.geo.nc * sizeof(int), st>>>(cv, b, layer, stage, flags,
                                                                                                  p_stride, T_a);
  }
  return cudaGetLastError();
}

}  // namespace wnw
