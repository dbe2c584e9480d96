// Token-granular prefill compression of fixed heads ("Prefill Compression"; retention per head from Eq. 1).
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

__device__ __forceinline__ int fixed_head_kv(const CacheView &cv, int layer, int f) {
  const Geometry &G = cv.geo;
  for (int h = 0; h < G.Hkv; ++h)
    if (cv.roles[layer * G.Hkv + h] == ROLE_FIXED && cv.role_idx[layer * G.Hkv + h] == f) return h;
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
  const int f = blockIdx.x, h = fixed_head_kv(cv, layer, f);
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
  const int f = blockIdx.x, h = fixed_head_kv(cv, layer, f);
  if (h < 0) return;
  const LayerInfo li = cv.layers[layer];
  const long long fh = (long long)b * G.F_tot + li.fixed_off + f;
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
  for (int s = threadIdx.x; s < G.S_max; s += TOK_THREADS)   // block s of the compact store holds min(nc, n - s*nc) rows
    cv.fixed_chunks[fh * G.S_max + s] = s < n_blk ? -(2 + min(G.nc, n - s * G.nc)) : -1;
  if (threadIdx.x == 0) { cv.fixed_n[fh] = n_blk; tok_n[fh] = n; }
}

// grid (S_max, fixed heads of the layer); block 128.  Fills block blockIdx.x of the head's compact store.
__global__ void __launch_bounds__(128) wnw_token_gather_kernel(const __grid_constant__ CacheView cv, int b, int layer,
                                                               const bf16 *stage, const int32_t *fixed_tok, int tok_cap,
                                                               const int32_t *tok_n) {
  const Geometry &G = cv.geo;
  const int blk = blockIdx.x, f = blockIdx.y, h = fixed_head_kv(cv, layer, f);
  if (h < 0) return;
  const LayerInfo li = cv.layers[layer];
  const long long fh = (long long)b * G.F_tot + li.fixed_off + f;
  const int n = tok_n[fh];
  if (blk * G.nc >= n) return;
  const int pieces = G.d / 8;
  const int32_t *pos = fixed_tok + fh * tok_cap;
  for (int kv = 0; kv < 2; ++kv) {
    const uint4 *src = reinterpret_cast<const uint4 *>(stage + anchor_off(G, 0, 0, h, kv));
    uint4 *dst = reinterpret_cast<uint4 *>(cv.fixed + fixed_off(G, li, b, f, kv) + (long long)blk * G.ncp * G.d);
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

cudaError_t launch_token_compress(const CacheView &cv, int b, int layer, int n_fixed, const bf16 *stage, const bf16 *q_text,
                                  int n_q, int T_t, int T_a, int seg, const float *retention_dev, int variant, float *work,
                                  float *p_tok, int32_t *flags, long long p_stride, int32_t *fixed_tok, int tok_cap,
                                  int32_t *tok_n, cudaStream_t st) {
  if (n_fixed <= 0 || T_a <= 0) return cudaSuccess;
  const size_t smem = (size_t)(cv.geo.d + TOK_THREADS / 32) * sizeof(float);
  wnw_token_score_kernel<<<n_fixed, TOK_THREADS, smem, st>>>(cv, b, layer, stage, q_text, n_q, T_t, T_a, work, p_tok, p_stride);
  wnw_token_select_kernel<<<n_fixed, TOK_THREADS, 0, st>>>(cv, b, layer, p_tok, p_stride, T_a, seg, retention_dev, variant, flags,
                                                          fixed_tok, tok_cap, tok_n);
  wnw_token_gather_kernel<<<dim3(cv.geo.S_max, n_fixed), 128, 0, st>>>(cv, b, layer, stage, fixed_tok, tok_cap, tok_n);
  return cudaGetLastError();
}

}  // namespace wnw
