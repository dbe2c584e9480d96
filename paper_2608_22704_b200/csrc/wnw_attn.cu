// Role-dispatched split-K decode attention with fused chunk-score partials (sm_100a).
//
// One launch per layer serves every KV head of every active sequence:
//   anchor heads : text + all audio (contiguous store); per 16-token granule the kernel also emits
//                  sum_tau 2^(s_tau - m) and the running max m, from which the tail kernel rebuilds the
//                  per-chunk softmax mass of Eq. 2 (Method section, "Decode-Step Score Aggregation");
//   tidal heads  : text + the chunks resident in the slot pool (gather by slot table);
//   fixed heads  : text + the compacted prefill subset.
// A CTA takes one work item = a granule range of one (sequence, KV head).  Each of its warps streams its
// own granules (16 tokens x d, K and V) through a private cp.async pipeline into XOR-swizzled shared
// memory and keeps a private online-softmax state; QK^T and PV run on mma.sync m16n8k16 with the g query
// heads of the group padded to the 16 rows of the tile (bf16 in, fp32 accumulate).  Warps merge through
// shared memory and the CTA writes one (m, l, o[g][d]) partial.
#include "wnw_internal.cuh"

namespace wnw {

constexpr int NW = 4;      // warps per CTA
constexpr int NSTAGE = 3;  // granules in flight per warp

int attn_warps() { return NW; }

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

struct GranDesc {
  const bf16 *k;   // first K row of the granule (V row = k + v_delta)
  int valid;       // visible tokens in the granule, 0 = nothing to do
  int score_idx;   // audio granule index for score partials, -1 = none
};

// Maps granule j of a head's virtual key space [text capacity | audio] to memory.
__device__ __forceinline__ GranDesc decode_granule(const CacheView &cv, const AttnArgs &a, const LayerInfo &li, int b, int h,
                                                   int role, int ridx, int j, int T_t, int T_a, int S_b) {
  const Geometry &G = cv.geo;
  GranDesc r;
  r.k = cv.text; r.valid = 0; r.score_idx = -1;
  if (j < G.n_tg) {
    const int tok0 = j * GR, v = T_t - tok0;
    if (v <= 0) return r;
    r.valid = v < GR ? v : GR;
    r.k = cv.text + text_off(G, b, a.layer, h, 0) + (long long)tok0 * G.d;
    return r;
  }
  const int ag = j - G.n_tg, ci = ag / G.gpc, off = (ag - ci * G.gpc) * GR;
  int c, store_row;
  const bf16 *base;
  if (role == ROLE_ANCHOR) {
    c = ci;
    base = a.anchor_base + anchor_off(G, a.anchor_seq_stride, b, a.anchor_head0 + ridx, 0);
    store_row = ci * G.nc + off;
  } else if (role == ROLE_TIDAL) {
    if (ci >= S_b) return r;
    c = cv.slot_chunk[((long long)b * G.L + a.layer) * G.S_max + ci];
    base = cv.pool + pool_off(G, li, b, ci, ridx, 0);
    store_row = off;
  } else {
    const long long fh = (long long)b * G.F_tot + li.fixed_off + ridx;
    c = ci < cv.fixed_n[fh] ? cv.fixed_chunks[fh * G.S_max + ci] : -1;
    base = cv.fixed + fixed_off(G, li, b, ridx, 0);
    store_row = ci * G.nc + off;
  }
  if (c < 0) return r;
  int len = T_a - c * G.nc;
  if (len > G.nc) len = G.nc;
  len -= off;
  if (len <= 0) return r;
  r.valid = len < GR ? len : GR;
  r.k = base + (long long)store_row * G.d;
  if (role == ROLE_ANCHOR && a.score_on) r.score_idx = ag;
  return r;
}

template <int D, bool G16>
__global__ void __launch_bounds__(NW * 32) wnw_attn_kernel(const __grid_constant__ CacheView cv,
                                                           const __grid_constant__ AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const Geometry &G = cv.geo;
  constexpr int ROWB = D * 2;             // bytes per K or V row
  constexpr int TILEB = GR * ROWB;        // bytes per K (or V) granule
  constexpr int PPR = D / 8;              // 16-byte pieces per row
  constexpr int KK = D / 16;              // k16 steps of QK^T; also pairs of n8 tiles of PV
  constexpr int NQ = G16 ? 4 : 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkItem it = a.items[blockIdx.x];
  const int b = a.active[it.i];
  const int g = G.g;
  const LayerInfo li = cv.layers[a.layer];
  int role = ROLE_ANCHOR, ridx = it.h;
  if (a.mode == ATTN_DECODE) {
    role = cv.roles[a.layer * G.Hkv + it.h];
    ridx = cv.role_idx[a.layer * G.Hkv + it.h];
  }
  const int T_t = cv.text_len[b] + a.has_new, T_a = cv.T_a[b], S_b = cv.S[b];
  long long v_delta_audio;
  if (role == ROLE_ANCHOR) v_delta_audio = (long long)G.T_a_pad * G.d;
  else if (role == ROLE_TIDAL) v_delta_audio = (long long)G.nc * G.d;
  else v_delta_audio = (long long)G.S_max * G.nc * G.d;
  const long long v_delta_text = (long long)G.T_cap_pad * G.d;

  __shared__ int2 ring[NW][NSTAGE];
  unsigned char *my_smem = smem + (size_t)warp * NSTAGE * 2 * TILEB;
  const uint32_t my_base = smem_u32(my_smem);

  // ---- Q fragments (rows >= g are zero padding) ----
  const int r0 = lane >> 2, cq = (lane & 3) * 2;
  uint32_t qa[KK][NQ];
  {
    const bf16 *qb = a.q + ((long long)it.i * G.Hq + (long long)it.h * g) * D;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      qa[kk][0] = r0 < g ? *reinterpret_cast<const uint32_t *>(qb + r0 * D + kk * 16 + cq) : 0u;
      qa[kk][1] = r0 < g ? *reinterpret_cast<const uint32_t *>(qb + r0 * D + kk * 16 + 8 + cq) : 0u;
      if (G16) {
        qa[kk][2] = r0 + 8 < g ? *reinterpret_cast<const uint32_t *>(qb + (r0 + 8) * D + kk * 16 + cq) : 0u;
        qa[kk][3] = r0 + 8 < g ? *reinterpret_cast<const uint32_t *>(qb + (r0 + 8) * D + kk * 16 + 8 + cq) : 0u;
      }
    }
  }

  float o[D / 8][4];
#pragma unroll
  for (int t = 0; t < D / 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  const int first = it.g0 + warp;
  const int n_my = first < it.g1 ? (it.g1 - first + NW - 1) / NW : 0;

  GranDesc blk;  // descriptor this lane decoded for the current block of 32 granules
  blk.k = cv.text; blk.valid = 0; blk.score_idx = -1;

  auto issue = [&](int n) {
    if (n < n_my) {
      if ((n & 31) == 0) {
        const int nn = n + lane;
        if (nn < n_my) blk = decode_granule(cv, a, li, b, it.h, role, ridx, first + nn * NW, T_t, T_a, S_b);
        else { blk.valid = 0; blk.score_idx = -1; }
      }
      const int src_lane = n & 31;
      const int valid = __shfl_sync(0xffffffffu, blk.valid, src_lane);
      const int sidx = __shfl_sync(0xffffffffu, blk.score_idx, src_lane);
      const unsigned long long kp = __shfl_sync(0xffffffffu, (unsigned long long)blk.k, src_lane);
      const int stage = n % NSTAGE;
      if (lane == 0) ring[warp][stage] = make_int2(valid, sidx);
      if (valid > 0) {
        const bf16 *k = reinterpret_cast<const bf16 *>(kp);
        const bool is_text = first + n * NW < G.n_tg;
        const bf16 *v = k + (is_text ? v_delta_text : v_delta_audio);
        const uint32_t sK = my_base + stage * 2 * TILEB, sV = sK + TILEB;
#pragma unroll
        for (int x = 0; x < GR * PPR / 32; ++x) {
          const int p = lane + 32 * x, row = p / PPR, pc = p % PPR;
          const int ok = row < valid;
          const int src_row = ok ? row : 0;
          const uint32_t dst = row * ROWB + ((pc ^ (row & 7)) << 4);
          cp_async16(sK + dst, k + (long long)src_row * D + pc * 8, ok ? 16 : 0);
          cp_async16(sV + dst, v + (long long)src_row * D + pc * 8, ok ? 16 : 0);
        }
      }
    }
    cp_async_commit();
  };

#pragma unroll
  for (int n = 0; n < NSTAGE - 1; ++n) issue(n);

  for (int n = 0; n < n_my; ++n) {
    cp_async_wait<NSTAGE - 2>();
    __syncwarp();
    const int stage = n % NSTAGE;
    const int2 rg = ring[warp][stage];
    const int valid = rg.x;
    if (valid > 0) {
      const uint32_t sK = my_base + stage * 2 * TILEB, sV = sK + TILEB;
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int mtx = lane >> 3, row = ((mtx >> 1) << 3) + (lane & 7);
        const uint32_t rowaddr = sK + row * ROWB;
#pragma unroll
        for (int kk = 0; kk < KK; ++kk) {
          uint32_t bk[4];
          const int piece = 2 * kk + (mtx & 1);
          ldsm_x4(bk, rowaddr + ((piece ^ (row & 7)) << 4));
          if (G16) {
            mma16816(s0, qa[kk][0], qa[kk][2], qa[kk][1], qa[kk][3], bk[0], bk[1]);
            mma16816(s1, qa[kk][0], qa[kk][2], qa[kk][1], qa[kk][3], bk[2], bk[3]);
          } else {
            mma16816(s0, qa[kk][0], 0u, qa[kk][1], 0u, bk[0], bk[1]);
            mma16816(s1, qa[kk][0], 0u, qa[kk][1], 0u, bk[2], bk[3]);
          }
        }
      }
      // ---- online softmax in log2 units, fp32; columns = tokens cq, cq+1, 8+cq, 9+cq ----
      const float sc = G.scale_log2;
      const bool k0 = cq < valid, k1 = cq + 1 < valid, k2 = cq + 8 < valid, k3 = cq + 9 < valid;
      float v0 = k0 ? s0[0] * sc : -INFINITY, v1 = k1 ? s0[1] * sc : -INFINITY;
      float v2 = k2 ? s1[0] * sc : -INFINITY, v3 = k3 ? s1[1] * sc : -INFINITY;
      float mx = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mn0 = fmaxf(m0, mx);
      const float al0 = exp2f(m0 - mn0);
      v0 = exp2f(v0 - mn0); v1 = exp2f(v1 - mn0); v2 = exp2f(v2 - mn0); v3 = exp2f(v3 - mn0);
      float rs0 = (v0 + v1) + (v2 + v3);
      rs0 += __shfl_xor_sync(0xffffffffu, rs0, 1);
      rs0 += __shfl_xor_sync(0xffffffffu, rs0, 2);
      l0 = l0 * al0 + rs0;
      m0 = mn0;
      uint32_t pa0 = pack_bf16(v0, v1), pa2 = pack_bf16(v2, v3), pa1 = 0u, pa3 = 0u;
      float al1 = 1.f, rs1 = 0.f;
      if (G16) {
        float w0 = k0 ? s0[2] * sc : -INFINITY, w1 = k1 ? s0[3] * sc : -INFINITY;
        float w2 = k2 ? s1[2] * sc : -INFINITY, w3 = k3 ? s1[3] * sc : -INFINITY;
        float my = fmaxf(fmaxf(w0, w1), fmaxf(w2, w3));
        my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 1));
        my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, 2));
        const float mn1 = fmaxf(m1, my);
        al1 = exp2f(m1 - mn1);
        w0 = exp2f(w0 - mn1); w1 = exp2f(w1 - mn1); w2 = exp2f(w2 - mn1); w3 = exp2f(w3 - mn1);
        rs1 = (w0 + w1) + (w2 + w3);
        rs1 += __shfl_xor_sync(0xffffffffu, rs1, 1);
        rs1 += __shfl_xor_sync(0xffffffffu, rs1, 2);
        l1 = l1 * al1 + rs1;
        m1 = mn1;
        pa1 = pack_bf16(w0, w1); pa3 = pack_bf16(w2, w3);
      }
      if (rg.y >= 0 && (lane & 3) == 0) {  // softmax-mass partial of this granule (fp32, before any bf16 rounding)
        float2 *ge = a.gran_em + ((long long)it.i * a.n_aq + (long long)ridx * g) * a.n_ag_max + rg.y;
        if (r0 < g) ge[(long long)r0 * a.n_ag_max] = make_float2(rs0, m0);
        if (G16 && r0 + 8 < g) ge[(long long)(r0 + 8) * a.n_ag_max] = make_float2(rs1, m1);
      }
#pragma unroll
      for (int t = 0; t < D / 8; ++t) {
        o[t][0] *= al0; o[t][1] *= al0;
        if (G16) { o[t][2] *= al1; o[t][3] *= al1; }
      }
      {
        const int mtx = lane >> 3, row = ((mtx & 1) << 3) + (lane & 7);
        const uint32_t rowaddr = sV + row * ROWB;
#pragma unroll
        for (int t2 = 0; t2 < KK; ++t2) {
          uint32_t bv[4];
          const int piece = 2 * t2 + (mtx >> 1);
          ldsm_x4_t(bv, rowaddr + ((piece ^ (row & 7)) << 4));
          mma16816(o[2 * t2], pa0, pa1, pa2, pa3, bv[0], bv[1]);
          mma16816(o[2 * t2 + 1], pa0, pa1, pa2, pa3, bv[2], bv[3]);
        }
      }
    }
    __syncwarp();
    issue(n + NSTAGE - 1);
  }
  cp_async_wait<0>();
  __syncthreads();

  // ---- merge the warps' partial states through shared memory ----
  float2 *red_ml = reinterpret_cast<float2 *>(smem);                           // [NW][16]
  float *red_o = reinterpret_cast<float *>(smem + NW * 16 * sizeof(float2));   // [NW][g][D]
  if ((lane & 3) == 0) {
    red_ml[warp * 16 + r0] = make_float2(m0, l0);
    red_ml[warp * 16 + r0 + 8] = make_float2(G16 ? m1 : -INFINITY, G16 ? l1 : 0.f);
  }
#pragma unroll
  for (int t = 0; t < D / 8; ++t) {
    if (r0 < g) *reinterpret_cast<float2 *>(red_o + ((size_t)warp * g + r0) * D + t * 8 + cq) = make_float2(o[t][0], o[t][1]);
    if (G16 && r0 + 8 < g)
      *reinterpret_cast<float2 *>(red_o + ((size_t)warp * g + r0 + 8) * D + t * 8 + cq) = make_float2(o[t][2], o[t][3]);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < g * D; idx += NW * 32) {
    const int row = idx / D, col = idx - row * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) M = fmaxf(M, red_ml[w * 16 + row].x);
    float acc = 0.f, L = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float2 ml = red_ml[w * 16 + row];
        const float f = exp2f(ml.x - M);   // a warp without work has m = -inf -> factor 0
        acc += red_o[((size_t)w * g + row) * D + col] * f;
        L += ml.y * f;
      }
    }
    a.part_o[((long long)blockIdx.x * g + row) * D + col] = acc;
    if (col == 0) a.part_ml[(long long)blockIdx.x * g + row] = make_float2(M, L);
  }
}

template <int D, bool G16>
static cudaError_t launch_t(const CacheView &cv, const AttnArgs &a, cudaStream_t st) {
  const size_t smem = (size_t)NW * NSTAGE * 2 * GR * D * 2;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(wnw_attn_kernel<D, G16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  wnw_attn_kernel<D, G16><<<a.n_items, NW * 32, smem, st>>>(cv, a);
  return cudaGetLastError();
}

cudaError_t launch_attn(const CacheView &cv, const AttnArgs &a, cudaStream_t st) {
  if (a.n_items <= 0) return cudaSuccess;
  const bool g16 = cv.geo.g > 8;
  if (cv.geo.d == 128) return g16 ? launch_t<128, true>(cv, a, st) : launch_t<128, false>(cv, a, st);
  if (cv.geo.d == 64) return g16 ? launch_t<64, true>(cv, a, st) : launch_t<64, false>(cv, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace wnw
