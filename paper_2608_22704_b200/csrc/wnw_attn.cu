// Role-dispatched split-K decode attention with fused chunk-score partials (sm_100a).
//
// One launch per layer serves every KV head of every active sequence:
//   anchor heads : text + all audio (contiguous store); per 16-token granule the kernel also emits
//                  sum_tau 2^(s_tau - m) and the running max m, from which the selection kernel rebuilds the
//                  per-chunk softmax mass of Eq. 2 (Method section, "Decode-Step Score Aggregation");
//   tidal heads  : text + the chunks resident in the slot pool (gather by slot table);
//   fixed heads  : text + the compacted prefill subset.
// A CTA takes one work item = a granule range of one (sequence, KV head), or walks a host-assigned list of them.  Each
// of its warps streams its own granules (16 tokens x d, K and V) through a private TMA pipeline (cp.async.bulk.tensor,
// 128-byte swizzle, one mbarrier per stage, issued by elected lanes) and keeps a private online-softmax state.  QK^T and PV
// run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) in transposed form, tokens on the M side of the tile and the group's
// query heads on N: S^T = K q^T, O^T = V^T P^T, so a group of up to 8 heads fills one n-tile without padding rows.  Warps
// merge through shared memory and the CTA writes the head's output, or one (m, l, o[g][d]) partial of a split head.
//
// The same launch also does the rest of the layer's step, with no further kernel and no host round trip:
//   - the warp that owns the text granule of the token being generated reads that row from k_new/v_new and
//     stores it into the text region (generated tokens are kept in full);
//   - the CTA that finishes a head last merges the head's split partials into bf16 outputs (log-sum-exp) and
//     publishes the head's final (max, denominator), which the selection kernel needs for the chunk scores.
// Chunk scoring, selection and recall are not needed by whatever consumes the attention output next, so they run
// in wnw_select_kernel / wnw_recall_kernel on a side stream (wnw_kernels.cu), off the critical path.
#include <cstring>
#include <type_traits>

#include <cuda_fp16.h>

#include "wnw_internal.cuh"
#include "wnw_tail.cuh"

namespace wnw {

constexpr int NW_LAT = 8;  // warps of a one-shot CTA (one work item each): 1 CTA per SM
constexpr int NW_THR = 4;  // warps of a persistent CTA (launches of more than one wave): several per SM, whose phases drift apart,
                           // so one CTA's prologue and merge overlap the others' streaming
// Granules in flight per warp, and persistent CTAs per SM.  Three stages and two 4-warp CTAs per SM are what was kept after
// measuring the alternative that shared memory allows, two-stage rings (exactly the pair a softmax step consumes) with
// three CTAs, i.e. twelve warps, per SM: 16 x 7500 tokens chained 0.417 -> 0.402 ms and overlapped 0.344 -> 0.360 ms,
// batch-32 ragged chained 1.31 -> 1.41 ms; two stages with two CTAs: 0.445, 0.355, 1.28 ms.  The macros are the sweep's.
#ifndef WNW_THR_CTAS_PER_SM
#define WNW_THR_CTAS_PER_SM 2
#endif
#ifndef WNW_NSTAGE_THR
#define WNW_NSTAGE_THR 3
#endif
constexpr int nstage_of(int nw) { return nw == NW_THR ? WNW_NSTAGE_THR : 3; }

int attn_warps(bool throughput) { return throughput ? NW_THR : NW_LAT; }
// Merge scratch of a CTA when it sits behind the stages instead of aliasing them: (m, l) and o of every warp.
static size_t attn_scratch_bytes(int nw, int g, int d) { return (size_t)nw * 128 + (size_t)nw * g * (d + 2) * 4; }
// Persistent CTAs an SM holds: what the shared memory allows (stages, alignment slack, merge scratch behind the stages,
// 1 KB the system keeps per CTA) up to what the kernel's register bound was compiled for.
int attn_persistent_ctas_per_sm(int g, int d) {
  const size_t per_cta = (size_t)NW_THR * nstage_of(NW_THR) * 2 * GR * d * 2 + 1024 + attn_scratch_bytes(NW_THR, g, d) + 512 + 1024;
  const int fit = (int)((228 * 1024) / per_cta);
  const int cap = g > 8 ? 2 : WNW_THR_CTAS_PER_SM;   // registers: the two-tile variant is compiled for two CTAs per SM
  return fit < 1 ? 1 : (fit > cap ? cap : fit);
}
// One-shot 8-warp CTAs can keep it there while everything fits the 227 KB a CTA may have.
bool attn_xpref_fits(int g, int d) {
  return (size_t)NW_LAT * nstage_of(NW_LAT) * 2 * GR * d * 2 + 1024 + attn_scratch_bytes(NW_LAT, g, d) + 512 <= 227 * 1024;
}


// Phase stamps for latency studies: compiled in only with -DWNW_PHASE_STAMPS (never in the product build).
#ifdef WNW_PHASE_STAMPS
#ifndef WNW_STAMP_CTAS
#define WNW_STAMP_CTAS 64
#endif
__device__ long long g_stamps[64 * 512 * 32];   // [layer * WNW_STAMP_CTAS + CTA of the layer's launch][phase], global-timer nanoseconds
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define STAMP(k) do { if (threadIdx.x == 0 && bid < WNW_STAMP_CTAS && a.layer * WNW_STAMP_CTAS < 64 * 512) g_stamps[(a.layer * WNW_STAMP_CTAS + bid) * 32 + (k)] = (long long)gtime(); } while (0)
#define GSTAMP(k) STAMP(k)
#define STAMPV(k, v) do { if (threadIdx.x == 0 && bid < WNW_STAMP_CTAS && a.layer * WNW_STAMP_CTAS < 64 * 512) g_stamps[(a.layer * WNW_STAMP_CTAS + bid) * 32 + (k)] = (long long)(v); } while (0)
extern "C" int wnw_debug_read_stamps(long long *host, int n_ctas) {
  return (int)cudaMemcpyFromSymbol(host, g_stamps, sizeof(long long) * 32 * n_ctas);
}
extern "C" int wnw_debug_clear_stamps() {
  static long long zeros[64 * 512 * 32];
  return (int)cudaMemcpyToSymbol(g_stamps, zeros, sizeof(zeros));
}
__device__ unsigned long long g_ktime[4 * 64 * 4];   // [step % 4][layer][start_min, trigger_max, end_max, unused], nanoseconds
#define KSTAMP_MIN(slot, k) do { if (threadIdx.x == 0) atomicMin(&g_ktime[(slot) * 4 + (k)], gtime()); } while (0)
#define KSTAMP_MAX(slot, k) do { if (threadIdx.x == 0) atomicMax(&g_ktime[(slot) * 4 + (k)], gtime()); } while (0)
extern "C" int wnw_debug_read_ktime(unsigned long long *host) { return (int)cudaMemcpyFromSymbol(host, g_ktime, sizeof(g_ktime)); }
extern "C" int wnw_debug_init_ktime() {
  static unsigned long long init[4 * 64 * 4];
  for (int i = 0; i < 4 * 64 * 4; ++i) init[i] = (i % 4 == 0) ? ~0ull : 0ull;
  return (int)cudaMemcpyToSymbol(g_ktime, init, sizeof(init));
}
#else
#define STAMP(k) do { } while (0)
#define GSTAMP(k) do { } while (0)
#define STAMPV(k, v) do { } while (0)
#define KSTAMP_MIN(slot, k) do { } while (0)
#define KSTAMP_MAX(slot, k) do { } while (0)
#endif

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// ---- mbarrier + TMA (every CTA fetches its own tiles) ----
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait: gives up after about a second of SM clocks and reports it instead of hanging.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > 2000000000ll) return false;
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n"
               ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
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

// Two e4m3 bytes (low 16 bits of x) as two fp16 numbers: one instruction, exact (every e4m3 value is an fp16 value).
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t x) {
  uint32_t h;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;\n" : "=r"(h) : "h"((unsigned short)x));
  return h;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// bf16 pair -> fp16 pair: exact for magnitudes inside fp16's normal range
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t x) { return pack_f16(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u)); }
__device__ __forceinline__ void mma16816_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct GranDesc {
  int row;         // first K row of the granule in its store's 2-D view [rows][d] (V row = row + v_delta)
  int meta;        // >= 0: visible tokens, known statically; -1: text granule, needs the text length; -2: needs `cid`;
                   // -3: needs `cid` and is not fetched at all when the slot is empty
  int cid;         // chunk id held by the slot / compact position (filled by a load that is not waited on here)
  int off;         // token offset of the granule inside its chunk
  int score_idx;   // audio granule index for score partials, -1 = none
  int ex;          // e4m3 tidal tier: K scale exponent | V scale exponent << 8 | 1 << 16 for a slot granule (filled with the metadata)
  int vis;         // visible rows, resolved with the first metadata of the descriptor's block of 32 granules
};

// Maps granule j of a head's virtual key space [text capacity | audio] to memory WITHOUT waiting on any global load:
// the row of every granule is static; what may be unknown yet is how many of its 16 rows are visible.
template <bool TB>
__device__ __forceinline__ GranDesc decode_granule(const CacheView &cv, const AttnArgs &a, const LayerInfo &li,
                                                   const WorkItem &it, int j, int table_parity) {
  const Geometry &G = cv.geo;
  GranDesc r;
  r.cid = -1; r.off = 0; r.score_idx = -1; r.ex = 0; r.vis = 0;
  if (j < G.n_tg) {
    const int tok0 = j * GR;
    r.row = (int)(text_off(G, it.b, a.layer, it.h, 0) / G.d) + tok0;
    r.meta = tok0 + GR <= it.T_hint ? GR : -1;
    return r;
  }
  const int ag = j - G.n_tg, ci = ag / G.gpc, off = (ag - ci * G.gpc) * GR;
  r.off = off;
  if (it.role == ROLE_ANCHOR) {
    r.row = (int)(anchor_off(G, a.anchor_seq_stride, it.b, a.anchor_head0 + it.ridx, 0) / G.d) + ci * G.ncp + off;
    int len = it.T_a - ci * G.nc;
    if (len > G.nc) len = G.nc;
    len -= off;
    r.meta = len <= 0 ? 0 : (len < GR ? len : GR);
    if (a.score_on) r.score_idx = ag;
  } else if (TB && it.role == ROLE_TIDAL && ci < it.S) {
    // token-granular permanent base: the first it.S units of the head are blocks of its compact store
    const int head = G.F_fix + li.tid_prefix + it.ridx;
    r.row = (int)(compact_off(G, it.b, head, 0) / G.d) + ci * G.ncp + off;
    r.cid = cv.fixed_chunks[((long long)it.b * G.F_tot + head) * G.FB + ci];
    r.meta = -2;
    r.score_idx = -2;               // marks the compact store (tensor map and K-to-V row distance differ from the pool's)
  } else if (it.role == ROLE_TIDAL) {
    const int slot = TB ? ci - it.S : ci;
    r.row = (int)(pool_off(G, li, it.b, slot, it.ridx, 0) / G.d) + off;
    r.cid = cv.slot_chunk[slot_table_off(G, table_parity, (long long)it.b * G.L + a.layer) + slot];
    // beyond the permanent slots a slot may be empty: its rows are fetched only if it is not
    r.meta = (TB || ci >= it.S) ? -3 : -2;
  } else {
    const long long fh = (long long)it.b * G.F_tot + li.fixed_off + it.ridx;
    r.row = (int)(fixed_off(G, li, it.b, it.ridx, 0) / G.d) + ci * G.ncp + off;
    r.cid = cv.fixed_chunks[fh * G.FB + ci];
    r.meta = -2;
  }
  return r;
}

// VAR 1 (TB): tidal heads keep a token-granular permanent base (their key space is [text | base blocks | dynamic slots]);
// VAR 2 (F8): the slot pool holds e4m3 bytes (one 16 x 128-byte box per K or V granule) with a power-of-two scale per
//   (chunk, head, K|V).  The bytes become fp16 fragments on their way from ldmatrix to mma.sync (one conversion per two
//   elements, exact), and the products with such a granule run on the fp16 form of mma.sync with q and P taken as fp16 (q
//   exactly while its elements lie in fp16's normal range; P in [0,1] with three more mantissa bits than bf16 gives it).  The
//   K scale multiplies the logits; the V scale enters the exponent of the granule's weights (see the softmax step).  The
//   default path (VAR 0) carries none of either variant's branches.
// bid: the CTA's index within its layer's launch (a launch may carry the CTAs of several layers back to back);
// inl: the layer's work items when they travel in the kernel parameters, else null (read from a.items).
template <int D, bool G16, int NW, int VAR>
__device__ __forceinline__ void attn_body(const CacheView &cv, const AttnArgs &a, const InlineItems *inl, const TmaMaps &maps,
                                          const int bid) {
  extern __shared__ unsigned char smem_raw[];
  // TMA boxes with the 128-byte swizzle must start on a 1024-byte boundary of the shared window
  unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const Geometry &G = cv.geo;
  constexpr int HALVES = D / 64;          // a K (or V) granule is HALVES boxes of 16 rows x 128 bytes
  constexpr int HALFB = GR * 128;         // bytes per box
  constexpr int TILEB = HALVES * HALFB;   // bytes per K (or V) granule
  constexpr int PPR = D / 8;              // 16-byte pieces per row
  constexpr int KK = D / 16;              // k16 steps of QK^T; also pairs of n8 tiles of PV
  constexpr int NQ = G16 ? 4 : 2;
  constexpr bool TB = VAR == 1, F8 = VAR == 2;
  constexpr int NSTAGE = nstage_of(NW);
  static_assert(!F8 || D == 128, "an e4m3 row must fill one 128-byte swizzle atom");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  STAMP(0);
  GSTAMP(14);
  // Programmatic dependent launch: the next layer's kernel may be scheduled right away.  A layer kernel touches only
  // its own layer's stores, partial buffers, counters and outputs, so consecutive layer kernels are independent and
  // may overlap as deeply as free SMs allow.  What later stream work relies on is that a completed kernel implies
  // that all earlier ones completed: one CTA waits for the predecessor right before it exits (pdl_finish).
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
#ifdef WNW_PHASE_STAMPS
  int kslot = 0;
#endif
  auto pdl_finish = [&]() {
    if (blockIdx.x == 0) {   // one CTA of the launch, whichever layer it serves
      asm volatile("griddepcontrol.wait;\n" ::: "memory");
      KSTAMP_MAX(kslot, 1);
    }
  };
  __shared__ int2 ring[NW][NSTAGE];                              // per stage: visible rows | loaded << 8, score index
  __shared__ __align__(8) unsigned long long bars[NW][NSTAGE];   // one mbarrier per stage, producer = consumer = this warp
  __shared__ int s_flag;
  const uint32_t my_base = smem_u32(smem + (size_t)warp * NSTAGE * 2 * TILEB);
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < NSTAGE; ++st) mbar_init(smem_u32(&bars[warp][st]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    fence_proxy_async();
  }
  __syncwarp();
  uint32_t phase_bits = 0;   // parity of each stage's barrier (carried across the CTA's work items)
  bool timed_out = false;
  const int g = G.g;
  const LayerInfo &li = a.li;
  // A CTA that serves several work items (short heads packed together) keeps its copy pipeline running across them:
  // while one item is merged, the first granules of the next are already in flight.  Its merge scratch then sits
  // behind the stages instead of aliasing them.
  const bool xpref = a.xpref != 0;

  // One work item per CTA when the launch fits the machine; otherwise a persistent CTA per SM walks the items the
  // host assigned to it (balanced by size), so no SM idles through a partial last wave.
  int q_begin = bid, q_end = bid + 1;
  if (a.cta_ranges) { q_begin = a.cta_ranges[bid]; q_end = a.cta_ranges[bid + 1]; }

  // What a warp needs to address the granules of one work item.
  struct Ctx {
    WorkItem it;
    int item_idx, T_t, v_delta_audio, first, n_my;
    int table_parity;     // which copy of the slot table this step reads (tidal items)
    int m_full, m_tail;   // token-granular base: positions of a full / of the last segment that live in the base already
    const int32_t *seg_kept;   // ... or, where they differ by segment (m_full < 0), the head's per-segment counts
    const CUtensorMap *map_audio;
  };
  // Replayed steps: the recall that refreshed this layer's slots ran outside the captured graph, possibly still
  // overlapping this step.  Bounded acquire-wait on the layer's epoch word before the first SLOT granule of a tidal item
  // is fetched; the text granules that precede it in the item go out first and hide the round trip.
  bool epoch_pending = false;
  auto wait_recall_epoch = [&]() {
    if (lane == 0) {
      const int expect = *a.expect_epoch;
      int seen;
      const long long t0 = clock64();
      for (;;) {
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];\n" : "=r"(seen) : "l"(a.wait_epoch) : "memory");
        if (seen >= expect) break;
        if (clock64() - t0 > 2000000000ll) { timed_out = true; break; }
      }
      asm volatile("fence.proxy.async.global;\n" ::: "memory");  // the slots are read by TMA (async proxy)
    }
    timed_out = __shfl_sync(0xffffffffu, (int)timed_out, 0) != 0;
    epoch_pending = false;
    if (warp == 0) STAMP(13);
  };
  int parity_b = -1, parity_v = 0;   // slot-table copy of the sequence whose tidal items this CTA is serving
  auto load_ctx = [&](Ctx &c, int qi, bool for_loads) {
    c.item_idx = a.cta_ranges ? a.order[qi] : qi;
    // short item lists travel in the kernel parameters: no global load before the first K/V load is issued
    c.it = (inl && a.n_items <= INLINE_ITEMS_MAX) ? inl->it[c.item_idx] : a.items[c.item_idx];
    c.T_t = cv.text_len[c.it.b] + a.has_new;
    if (c.it.role == ROLE_ANCHOR) { c.v_delta_audio = G.T_a_pad; c.map_audio = &maps.anchor; }       // rows between a
    else if (c.it.role == ROLE_TIDAL) { c.v_delta_audio = G.ncp; c.map_audio = &maps.pool; }          // granule's K and
    else { c.v_delta_audio = G.FB * G.ncp; c.map_audio = &maps.fixed; }                            // V rows
    c.m_full = c.m_tail = 0;
    if (c.it.role == ROLE_TIDAL && cv.steps && c.it.b != parity_b) {   // once per sequence a CTA serves, not per item
      parity_b = c.it.b;
      parity_v = (int)(cv.steps[c.it.b] & 1);
    }
    c.table_parity = c.it.role == ROLE_TIDAL ? parity_v : 0;
    if (TB && c.it.role == ROLE_TIDAL) {
      const int2 m = cv.tok_m[((long long)c.it.b * G.L + a.layer) * G.Hkv + c.it.h];
      c.m_full = m.x; c.m_tail = m.y;
      c.seg_kept = cv.seg_kept + ((long long)c.it.b * cv.tid_total + li.tid_prefix + c.it.ridx) * G.C_max;
    }
    c.first = c.it.g0 + warp;
    c.n_my = c.first < c.it.g1 ? (c.it.g1 - c.first + NW - 1) / NW : 0;
    if (for_loads) epoch_pending = a.wait_epoch != nullptr && c.it.role == ROLE_TIDAL;   // see wait_recall_epoch
  };
  const int v_delta_text = G.T_cap_pad;

  // ---- producer side of the per-warp pipeline: (prod, p_n) is the next granule to fetch, seq_p its stage sequence ----
  Ctx prod;
  prod.n_my = 0;   // loaded by the first work item before anything is produced
  int p_n = 0;
  uint32_t seq_p = 0, seq_c = 0;
  GranDesc blk;  // descriptor this lane decoded for the producer's current block of 32 granules
  blk.row = 0; blk.meta = 0; blk.cid = -1; blk.off = 0; blk.score_idx = -1; blk.ex = 0; blk.vis = 0;

  // Visible rows of a granule once its metadata has arrived.
  auto visible = [&](const Ctx &c, int meta, int cid, int off, int j) -> int {
    if (meta >= 0) return meta;
    int len;
    if (meta == -1) len = c.T_t - j * GR;
    else {
      if (cid == -1) return 0;
      if (cid < -1) len = -cid - 2;   // a block of a token-compacted fixed head: the entry carries its row count
      else {
        len = c.it.T_a - cid * G.nc;
        if (len > G.nc) len = G.nc;
        // token base: a fetched segment holds its complement first; the last segment has its own count
        if (TB) len -= c.m_full < 0 ? c.seg_kept[cid] : (c.it.T_a - cid * G.nc > G.nc) ? c.m_full : c.m_tail;
      }
      len -= off;
    }
    return len <= 0 ? 0 : (len < GR ? len : GR);
  };
  // Queues the TMA copies of granule n of item c (K and V, all 16 rows) into stage seq % NSTAGE.  Granules with a static
  // row are fetched before anyone knows how many of their rows are visible (the stores hold finite data everywhere;
  // masked columns get probability 0); only text granules beyond the host's lower bound wait for the text length.
  // Returns whether a copy was queued.
  auto issue_copy = [&](const Ctx &c, int n, uint32_t seq) -> bool {
    if ((n & 31) == 0) {
      const int nn = n + lane;
      if (nn < c.n_my) blk = decode_granule<TB>(cv, a, li, c.it, c.first + nn * NW, c.table_parity);
      else { blk.meta = 0; blk.cid = -1; blk.score_idx = -1; blk.ex = 0; }
#ifdef WNW_PHASE_STAMPS
      if (n == 0 && blk.row >= 0) STAMP(12);
#endif
    }
    const int src_lane = n & 31;
    const int meta = __shfl_sync(0xffffffffu, blk.meta, src_lane);
    const int row = __shfl_sync(0xffffffffu, blk.row, src_lane);
    const int j = c.first + n * NW;
    const bool is_text = j < G.n_tg;
    // a block of a tidal head's permanent token base: compact store, never touched by the recall
    const bool base_blk = TB && __shfl_sync(0xffffffffu, blk.score_idx, src_lane) == -2;
    if (epoch_pending && !is_text && !base_blk) wait_recall_epoch();
    bool load = meta != 0;
    if (meta == -1) load = visible(c, -1, 0, 0, j) > 0;  // waits for the text length
    if (meta == -3) load = __shfl_sync(0xffffffffu, blk.cid, src_lane) >= 0;  // waits for the table entry
    // The boxes of a granule (K and V, HALVES each) are issued by as many lanes at once, one box per lane: lane = 2 * half + (V).
    // The stage's barrier cannot complete before lane 0 has arrived with the byte count, whichever copy lands first.
    const bool f8g = F8 && !is_text && c.it.role == ROLE_TIDAL;   // an e4m3 granule: one box of 16 rows x 128 bytes each for K and V
    if (load && lane < (f8g ? 2 : 2 * HALVES)) {
      const int stage = (int)(seq % NSTAGE);
      const uint32_t bar = smem_u32(&bars[warp][stage]);
      const CUtensorMap *map = is_text ? &maps.text : (base_blk ? &maps.fixed : c.map_audio);
      const int v_delta = is_text ? v_delta_text : (base_blk ? G.FB * G.ncp : c.v_delta_audio);
      const int hf = lane >> 1, isv = lane & 1;
      fence_proxy_async();  // the stage was last read through the generic proxy (ldmatrix)
      if (lane == 0) mbar_expect_tx(bar, f8g ? 2 * HALFB : 2 * TILEB);
      tma_load_2d(my_base + stage * 2 * TILEB + isv * TILEB + hf * HALFB, map, hf * 64, row + isv * v_delta, bar);
    }
    return load;
  };
  // Publishes (visible rows, loaded, score index) of granule n of item c for the compute step; may wait for the
  // metadata loads.
  auto issue_meta = [&](const Ctx &c, int n, uint32_t seq, bool loaded) {
    const int src_lane = n & 31;
    // every lane resolves its own granule of the block once (this is where the table entries and the text length are waited for)
    if (src_lane == 0) blk.vis = visible(c, blk.meta, blk.cid, blk.off, c.first + (n + lane) * NW);
    const int valid = __shfl_sync(0xffffffffu, blk.vis, src_lane);
    const int sidx = __shfl_sync(0xffffffffu, blk.score_idx, src_lane);
    int ex = 0;
    if (F8) {
      // the scales of the chunks this block of 32 granules touches: one load per lane and block, once the chunk ids are there
      if (src_lane == 0) {
        blk.ex = 0;
        if (n + lane < c.n_my && c.first + (n + lane) * NW >= G.n_tg && c.it.role == ROLE_TIDAL && blk.cid >= 0)
          blk.ex = 0x10000 | *reinterpret_cast<const unsigned short *>(
                                 cv.kv_exp + kv_exp_off(G, cv.tid_total, c.it.b, li.tid_prefix + c.it.ridx, blk.cid));
      }
      ex = __shfl_sync(0xffffffffu, blk.ex, src_lane);
    }
    // x: visible rows | copy queued << 8 | e4m3 granule << 9 | K exponent << 16 | V exponent << 24
    if (lane == 0) ring[warp][seq % NSTAGE] = make_int2(valid | (loaded ? 256 : 0) | ((ex >> 16) << 9) | (int)(((unsigned)ex & 0xffffu) << 16), sidx);
  };
  // Fetches the producer's next granule, moving on to the CTA's next work item when this warp has none left in the
  // current one (only when the pipeline runs across items).
  int p_qi = q_begin;
  auto produce = [&]() {
    while (p_n >= prod.n_my) {
      if (!xpref || p_qi + 1 >= q_end) return;
      ++p_qi;
      load_ctx(prod, p_qi, true);
      p_n = 0;
    }
    const bool ld = issue_copy(prod, p_n, seq_p);
    issue_meta(prod, p_n, seq_p, ld);
    ++p_n; ++seq_p;
  };

  uint32_t prewaited = 0;   // stages whose bytes have been waited for ahead of the inputs (chained layers)
  for (int qi = q_begin; qi < q_end; ++qi) {
  // without a scratch region of its own the merge below reuses the stages: the previous item's merge must be done
  if (qi > q_begin && !xpref) __syncthreads();
  const bool arm = !xpref || qi == q_begin;   // (re)start the pipeline at this item
  Ctx cc;
  if (arm) {
    p_qi = qi; p_n = 0;
    load_ctx(prod, qi, true);
    cc = prod;
  } else {
    load_ctx(cc, qi, false);
  }
  const WorkItem &it = cc.it;
  const int item_idx = cc.item_idx;
  if (cv.step_snap && it.h == 0 && it.g0 == 0 && threadIdx.x == 0 && a.mode != ATTN_PREFILL)   // (no cache state behind the
    cv.step_snap[(long long)it.b * G.L + a.layer] = cv.steps[it.b];                            //  allocation-free entry)
  const int b = it.b, ridx = it.ridx, T_t = cc.T_t;
  const int first = cc.first, n_my = cc.n_my;
#ifdef WNW_PHASE_STAMPS
  if (it.g0 >= 0) STAMP(10);
  kslot = (int)((cv.steps[b] & 3) * 64 + a.layer);
  KSTAMP_MIN(kslot, 0);
#endif
  // the first copies go out before anything else is read; their metadata follows the Q loads
  bool pro_loaded[NSTAGE];
  int n_pro = 0;
  if (arm) {
#pragma unroll
    for (int n = 0; n < NSTAGE; ++n)
      if (n < n_my) { pro_loaded[n] = issue_copy(prod, n, seq_p + n); n_pro = n + 1; }
  }
  STAMP(1);
  // Chained layers: while the preceding work still runs, this warp resolves the metadata of the granules it has queued,
  // waits for their bytes and clears masked V rows; none of it depends on that work.  What is left behind the wait is the
  // query load, the arithmetic and the merge.
  const bool early = arm && a.wait_inputs && qi == q_begin;
  if (early) {
#pragma unroll
    for (int n = 0; n < NSTAGE; ++n)
      if (n < n_pro) issue_meta(prod, n, seq_p + n, pro_loaded[n]);
    __syncwarp();
#pragma unroll
    for (int n = 0; n < NSTAGE; ++n)
      if (n < n_pro && !timed_out) {
        const int stage = (int)((seq_p + n) % NSTAGE);
        const int2 rg = ring[warp][stage];
        const int valid = rg.x & 255;
        if (rg.x & 256) {
          if (!mbar_wait(smem_u32(&bars[warp][stage]), (phase_bits >> stage) & 1u)) timed_out = true;
          else { phase_bits ^= 1u << stage; prewaited |= 1u << stage; }
        }
        if (valid > 0 && valid < GR && !timed_out) {
          const uint32_t sVz = my_base + stage * 2 * TILEB + TILEB;
          for (int r = valid + (lane >> 3); r < GR; r += 4)
#pragma unroll
            for (int hf = 0; hf < HALVES; ++hf)
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};\n" ::"r"(sVz + hf * HALFB + r * 128 + ((lane & 7) << 4)), "r"(0u) : "memory");
        }
      }
    p_n = n_pro; seq_p += n_pro;
    // the consumer takes two granules at a time and counts on the producer being a full ring ahead: an item shorter than
    // the pipeline is topped up from the items that follow, here as on the ordinary path
    if (xpref)
      for (int n = n_pro; n < NSTAGE; ++n) produce();
  }

  // Chained layers: the cache loads above never depend on the preceding work, the query and the new token's K/V do.
  // Their lines are asked into L2 ahead of the wait (L2 is where the preceding work's stores land, so nothing stale can
  // be read from it); the loads after the wait go past L1.
  if (a.wait_inputs && qi == q_begin) {
    const char *qline = reinterpret_cast<const char *>(a.q + ((long long)it.i * G.Hq + (long long)it.h * g) * D);
    if (threadIdx.x * 128 < g * D * 2) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(qline + threadIdx.x * 128));
    if (a.has_new && threadIdx.x < 2) {
      const bf16 *nb = (threadIdx.x ? a.v_new : a.k_new) + ((long long)it.i * G.Hkv + it.h) * D;
      asm volatile("prefetch.global.L2 [%0];\n" ::"l"(nb));
      if (D * 2 > 128) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(reinterpret_cast<const char *>(nb) + 128));
    }
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
  }
  STAMP(6);
  // ---- Q fragments (the B operand of S^T = K q^T; heads >= g are zero columns); loaded after the first K/V copies are in flight ----
  const int r0 = lane >> 2, cq = (lane & 3) * 2;
  uint32_t qa[KK][NQ];
  {
    const bf16 *qb = a.q + ((long long)it.i * G.Hq + (long long)it.h * g) * D;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      qa[kk][0] = r0 < g ? __ldcg(reinterpret_cast<const uint32_t *>(qb + r0 * D + kk * 16 + cq)) : 0u;
      qa[kk][1] = r0 < g ? __ldcg(reinterpret_cast<const uint32_t *>(qb + r0 * D + kk * 16 + 8 + cq)) : 0u;
      if (G16) {
        qa[kk][2] = r0 + 8 < g ? __ldcg(reinterpret_cast<const uint32_t *>(qb + (r0 + 8) * D + kk * 16 + cq)) : 0u;
        qa[kk][3] = r0 + 8 < g ? __ldcg(reinterpret_cast<const uint32_t *>(qb + (r0 + 8) * D + kk * 16 + 8 + cq)) : 0u;
      }
    }
  }
  uint32_t qh[F8 ? KK : 1][NQ];   // the query as fp16, for the products with e4m3 granules
  if constexpr (F8) {
    if (it.role == ROLE_TIDAL) {
#pragma unroll
      for (int kk = 0; kk < KK; ++kk)
#pragma unroll
        for (int x = 0; x < NQ; ++x) qh[kk][x] = bf16x2_to_f16x2(qa[kk][x]);
    }
  }
  STAMP(16);
  if (arm && !early) {
#pragma unroll
    for (int n = 0; n < NSTAGE; ++n) {
      if (n < n_pro) issue_meta(prod, n, seq_p + n, pro_loaded[n]);
      if (n == 0) STAMP(23);
    }
    p_n = n_pro; seq_p += n_pro;
    if (xpref)   // an item shorter than the pipeline: top up from the items that follow
      for (int n = n_pro; n < NSTAGE; ++n) produce();
  }

  // ---- per-warp state, transposed: tokens on the M side of the tile, query heads on N ----
  // S^T[token][head] = K q^T and O^T[d][head] = V^T P^T: an m16n8k16 tile then holds 16 tokens x 8 query heads, so a
  // group of up to 8 heads fills it with no padding rows (16 heads: two n-tiles) and the accumulators are a quarter of
  // the [head][d] form's.  A lane owns heads hq = nt*8 + cq + {0,1} of every n-tile: for S^T at tokens r0 and r0+8 of
  // the granule, for O^T at d = 16 t + r0 and 16 t + r0 + 8.
  constexpr int NTN = G16 ? 2 : 1;
  float oT[NTN][D / 16][4];
  float mrun[NTN][2], lrun[NTN][2];   // running max (log2 units, equal in the lanes that share a head) and this lane's share of the denominator
#pragma unroll
  for (int nt = 0; nt < NTN; ++nt) {
#pragma unroll
    for (int t = 0; t < D / 16; ++t) oT[nt][t][0] = oT[nt][t][1] = oT[nt][t][2] = oT[nt][t][3] = 0.f;
    mrun[nt][0] = mrun[nt][1] = -INFINITY; lrun[nt][0] = lrun[nt][1] = 0.f;
  }
  const float sc = G.scale_log2;

  // One step of the online softmax over NU granules (16 or 32 tokens) that sit in the given stages: two granules give the
  // warp two independent chains of everything (and one max/rescale for both).
  // fmt (e4m3 tier only): per granule 0 = bf16 tile, else 1 | K exponent << 16 | V exponent << 24 (as in the ring entry >> 9)
  auto step = [&](auto nu_tag, const uint32_t (&sKs)[2], const uint32_t (&sVs)[2], const int (&valids)[2], const int (&sidxs)[2],
                  const int (&fmt)[2]) {
    constexpr int NU = decltype(nu_tag)::value;
    float sT[NU][NTN][4];
    // e4m3 granules: the K scale 2^eK multiplies the logits.  The V scale 2^eV is carried in the exponent: the granule's
    // logits are shifted by eV for the running maximum and the weights, so that P = 2^(s + eV - m) <= 1 multiplies the raw
    // e4m3 values of V, and the denominator takes each weight times 2^-eV.  The triple (m, l, o) stays consistent for every
    // merge: both l and o are relative to the same m, whatever m is.
    float scu[NU], vshift[NU], vinv[NU];
#pragma unroll
    for (int u = 0; u < NU; ++u) {
      scu[u] = sc; vshift[u] = 0.f; vinv[u] = 1.f;
      if (F8 && (fmt[u] & 1)) {
        scu[u] = sc * exp2f((float)(int8_t)((fmt[u] >> 7) & 0xff));
        vshift[u] = (float)(int8_t)((fmt[u] >> 15) & 0xff);
        vinv[u] = exp2f(-vshift[u]);
      }
    }
    {
      float sO[NU][NTN][4];   // odd k-steps: shorter dependent mma chains
#pragma unroll
      for (int u = 0; u < NU; ++u)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) sT[u][nt][e] = sO[u][nt][e] = 0.f;
      const int mtx = lane >> 3;
      // A lane's ldmatrix row address inside a 16 x 128-byte box with the 128-byte swizzle: row * 128 + ((piece ^ row % 8) << 4),
      // piece = 2 * kk + (0 or 1 by lane).  The lane's part, row * 128 + (((0 or 1) ^ row % 8) << 4), is a constant of the
      // lane; a k-step then costs one XOR with an immediate (stages start on 1024-byte boundaries, so the base adds in freely).
      const uint32_t lane_k = (uint32_t)((((mtx >> 1) << 3) + (lane & 7)) * 128 + (((mtx & 1) ^ (lane & 7)) << 4));
      auto qk_bf16 = [&](int kk, int u) {
        uint32_t bk[4];   // K rows 0-7 | 8-15 of the granule x d 0-7 | 8-15 of the k-step: the A operand's four quadrants
        ldsm_x4(bk, ((sKs[u] + lane_k) ^ (uint32_t)(((2 * kk) & 7) << 4)) + (kk >> 2) * HALFB);
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt)
          mma16816((kk & 1) ? sO[u][nt] : sT[u][nt], bk[0], bk[2], bk[1], bk[3], qa[kk][2 * nt], qa[kk][2 * nt + 1]);
      };
      if constexpr (!F8) {
#pragma unroll
        for (int kk = 0; kk < KK; ++kk)
#pragma unroll
          for (int u = 0; u < NU; ++u) qk_bf16(kk, u);
      } else {
#pragma unroll
        for (int u = 0; u < NU; ++u) {
          if (fmt[u] & 1) {
            // e4m3 tile: rows of 128 bytes; one ldmatrix.x4 brings rows 0-7 | 8-15 x the 16-byte groups 2p | 2p+1, i.e. two
            // k-steps; a lane's four bytes are the elements 2t, 2t+1, 2t+8, 2t+9 of the group (e4m3_store_pos)
            const uint32_t lane_k8 = (uint32_t)((((mtx & 1) << 3) + (lane & 7)) * 128 + (((mtx >> 1) ^ (lane & 7)) << 4));
#pragma unroll
            for (int p = 0; p < KK / 2; ++p) {
              uint32_t bk[4];
              ldsm_x4(bk, (sKs[u] + lane_k8) ^ (uint32_t)((2 * p) << 4));
#pragma unroll
              for (int hk = 0; hk < 2; ++hk) {
                const uint32_t a0 = e4m3x2_to_f16x2(bk[2 * hk]), a1 = e4m3x2_to_f16x2(bk[2 * hk + 1]);
                const uint32_t a2 = e4m3x2_to_f16x2(bk[2 * hk] >> 16), a3 = e4m3x2_to_f16x2(bk[2 * hk + 1] >> 16);
#pragma unroll
                for (int nt = 0; nt < NTN; ++nt)
                  mma16816_f16(hk ? sO[u][nt] : sT[u][nt], a0, a1, a2, a3, qh[2 * p + hk][2 * nt], qh[2 * p + hk][2 * nt + 1]);
              }
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < KK; ++kk) qk_bf16(kk, u);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < NU; ++u)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) sT[u][nt][e] += sO[u][nt][e];
    }
    STAMP(25);
    // ---- online softmax per query head (a column of S^T), log2 units, fp32 ----
    uint32_t pb[NU][NTN][2];   // P^T as the B operand of the PV product: tokens 0-7 | 8-15 of the granule x this lane's head
#pragma unroll
    for (int nt = 0; nt < NTN; ++nt) {
      float v[NU][4];
      float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        const bool lo = r0 < valids[u], hi = r0 + 8 < valids[u];
        v[u][0] = lo ? fmaf(sT[u][nt][0], scu[u], vshift[u]) : -INFINITY; v[u][1] = lo ? fmaf(sT[u][nt][1], scu[u], vshift[u]) : -INFINITY;
        v[u][2] = hi ? fmaf(sT[u][nt][2], scu[u], vshift[u]) : -INFINITY; v[u][3] = hi ? fmaf(sT[u][nt][3], scu[u], vshift[u]) : -INFINITY;
        mxA = fmaxf(mxA, fmaxf(v[u][0], v[u][2])); mxB = fmaxf(mxB, fmaxf(v[u][1], v[u][3]));
      }
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, sh));
        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, sh));
      }
      const float mnA = fmaxf(mrun[nt][0], mxA), mnB = fmaxf(mrun[nt][1], mxB);   // finite: the step has a visible token
      const float alA = exp2f(mrun[nt][0] - mnA), alB = exp2f(mrun[nt][1] - mnB);
      mrun[nt][0] = mnA; mrun[nt][1] = mnB;
      float addA = 0.f, addB = 0.f;
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        v[u][0] = exp2f(v[u][0] - mnA); v[u][2] = exp2f(v[u][2] - mnA);
        v[u][1] = exp2f(v[u][1] - mnB); v[u][3] = exp2f(v[u][3] - mnB);
        float eA = v[u][0] + v[u][2], eB = v[u][1] + v[u][3];
        if constexpr (F8) { addA += eA * vinv[u]; addB += eB * vinv[u]; }
        else { addA += eA; addB += eB; }
        if (sidxs[u] >= 0) {   // softmax-mass partial of this granule (fp32, before any bf16 rounding): anchor-like heads only
#pragma unroll
          for (int sh = 4; sh <= 16; sh <<= 1) {
            eA += __shfl_xor_sync(0xffffffffu, eA, sh);
            eB += __shfl_xor_sync(0xffffffffu, eB, sh);
          }
          if (r0 == 0) {
            const int hq = nt * 8 + cq;
            float2 *ge = a.gran_em + ((long long)it.i * a.n_aq + (long long)ridx * g + hq) * a.n_ag_max + sidxs[u];
            if (hq < g) ge[0] = make_float2(eA, mnA);
            if (hq + 1 < g) ge[a.n_ag_max] = make_float2(eB, mnB);
          }
        }
        // P^T tile [token][head] -> [head][token]: what the PV product wants in its B operand
        uint32_t p01, p23;
        if (F8 && (fmt[u] & 1)) {   // fp16 weights for the fp16 product with an e4m3 granule
          p01 = pack_f16(v[u][0], v[u][1]); p23 = pack_f16(v[u][2], v[u][3]);
        } else {
          p01 = pack_bf16(v[u][0], v[u][1]); p23 = pack_bf16(v[u][2], v[u][3]);
        }
        asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(pb[u][nt][0]) : "r"(p01));
        asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(pb[u][nt][1]) : "r"(p23));
      }
      lrun[nt][0] = lrun[nt][0] * alA + addA; lrun[nt][1] = lrun[nt][1] * alB + addB;
#pragma unroll
      for (int t = 0; t < D / 16; ++t) { oT[nt][t][0] *= alA; oT[nt][t][1] *= alB; oT[nt][t][2] *= alA; oT[nt][t][3] *= alB; }
    }
    STAMP(26);
    {
      const int mtx = lane >> 3;
      const uint32_t lane_v = (uint32_t)((((mtx & 1) << 3) + (lane & 7)) * 128 + (((mtx >> 1) ^ (lane & 7)) << 4));   // as lane_k above
      auto pv_bf16 = [&](int t2, int u) {
        uint32_t bv[4];   // V^T: tokens 0-7 | 8-15 x d 0-7 | 8-15 of the 16-wide d tile, transposed on the way out of shared memory
        ldsm_x4_t(bv, ((sVs[u] + lane_v) ^ (uint32_t)(((2 * t2) & 7) << 4)) + (t2 >> 2) * HALFB);
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt) mma16816(oT[nt][t2], bv[0], bv[2], bv[1], bv[3], pb[u][nt][0], pb[u][nt][1]);
      };
      if constexpr (!F8) {
#pragma unroll
        for (int t2 = 0; t2 < KK; ++t2)
#pragma unroll
          for (int u = 0; u < NU; ++u) pv_bf16(t2, u);
      } else {
#pragma unroll
        for (int u = 0; u < NU; ++u) {
          if (fmt[u] & 1) {
            // e4m3 tile, transposed in 16-bit units: a lane gets tokens 2t, 2t+1 of the unit (bytes 2r, 2r+1 of the group) that
            // holds the elements r and r+8 of the d-tile: one byte permute sorts them into the two accumulator rows
#pragma unroll
            for (int p = 0; p < KK / 2; ++p) {
              uint32_t bv[4];   // tokens 0-7 | 8-15 x the 16-byte groups 2p | 2p+1 (two d-tiles)
              ldsm_x4_t(bv, (sVs[u] + lane_v) ^ (uint32_t)((2 * p) << 4));
#pragma unroll
              for (int hk = 0; hk < 2; ++hk) {
                const uint32_t x0 = __byte_perm(bv[2 * hk], 0, 0x3120), x1 = __byte_perm(bv[2 * hk + 1], 0, 0x3120);
                const uint32_t a0 = e4m3x2_to_f16x2(x0), a1 = e4m3x2_to_f16x2(x0 >> 16);
                const uint32_t a2 = e4m3x2_to_f16x2(x1), a3 = e4m3x2_to_f16x2(x1 >> 16);
#pragma unroll
                for (int nt = 0; nt < NTN; ++nt) mma16816_f16(oT[nt][2 * p + hk], a0, a1, a2, a3, pb[u][nt][0], pb[u][nt][1]);
              }
            }
          } else {
#pragma unroll
            for (int t2 = 0; t2 < KK; ++t2) pv_bf16(t2, u);
          }
        }
      }
    }
  };

  STAMP(17);
  const int new_j = a.has_new ? (T_t - 1) / GR : -1;   // the text granule that takes the row of the token being generated
  for (int n = 0; n < n_my && !timed_out;) {
    __syncwarp();
    // up to two granules per step; a granule with nothing visible (an empty slot, text capacity not yet written) is passed over
    const int cnt = n + 1 < n_my ? 2 : 1;
    uint32_t sKs[2] = {0u, 0u}, sVs[2] = {0u, 0u};
    int valids[2] = {0, 0}, sidxs[2] = {-1, -1}, fmt[2] = {0, 0};
    int nu = 0, adv = 0;
    if (n == 0) STAMP(18);
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (u < cnt && !timed_out) {
        const int stage = (int)((seq_c + u) % NSTAGE);
        const int2 rg = ring[warp][stage];
        const int valid = rg.x & 255;
        const bool pre = (prewaited >> stage) & 1u;   // waited for (and masked rows cleared) ahead of the inputs
        prewaited &= ~(1u << stage);
        if ((rg.x & 256) && !pre) {  // a copy was queued for this stage: wait for its bytes (bounded)
          if (!mbar_wait(smem_u32(&bars[warp][stage]), (phase_bits >> stage) & 1u)) timed_out = true;
          else phase_bits ^= 1u << stage;
        }
        if (!timed_out) ++adv;
        if (n == 0 && u == 0) STAMP(24);
        if (valid > 0 && !timed_out) {
          const uint32_t sK = my_base + stage * 2 * TILEB, sV = sK + TILEB;
          // the row of the token being generated: take it from k_new/v_new and store it into the text region
          const int j = first + (n + u) * NW;
          if (j == new_j) {
            const int nr = (T_t - 1) - j * GR;
            if (lane < 2 * PPR) {
              const int kv = lane / PPR, pc = lane - kv * PPR;
              const long long noff = ((long long)it.i * G.Hkv + it.h) * D + pc * 8;
              const uint4 val = __ldcg(reinterpret_cast<const uint4 *>((kv ? a.v_new : a.k_new) + noff));
              *reinterpret_cast<uint4 *>(cv.text + text_off(G, b, a.layer, it.h, kv) + (long long)(T_t - 1) * D + pc * 8) = val;
              const uint32_t dst = (kv ? sV : sK) + (pc >> 3) * HALFB + nr * 128 + (((pc & 7) ^ (nr & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};\n" ::"r"(dst), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
            }
          }
          if (valid < GR && !pre) {
            // rows past the visible ones get probability 0, but 0 x NaN is NaN and a caller-owned buffer (the allocation-free
            // entry) may hold anything there: clear those V rows (a masked K row only spoils logits that are replaced anyway)
            for (int r = valid + (lane >> 3); r < GR; r += 4)
#pragma unroll
              for (int hf = 0; hf < HALVES; ++hf)
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};\n" ::"r"(sV + hf * HALFB + r * 128 + ((lane & 7) << 4)), "r"(0u) : "memory");
          }
          if (nu == 0) { sKs[0] = sK; sVs[0] = sV; valids[0] = valid; sidxs[0] = rg.y; fmt[0] = rg.x >> 9; }
          else { sKs[1] = sK; sVs[1] = sV; valids[1] = valid; sidxs[1] = rg.y; fmt[1] = rg.x >> 9; }
          ++nu;
        }
      }
    }
    __syncwarp();
    if (n == 0) STAMP(7);
    if (timed_out) { seq_c += adv; break; }   // the stages whose bytes never came are drained (bounded) before the CTA ends
    {
      if (nu == 2) step(std::integral_constant<int, 2>{}, sKs, sVs, valids, sidxs, fmt);
      else if (nu == 1) step(std::integral_constant<int, 1>{}, sKs, sVs, valids, sidxs, fmt);
    }
    __syncwarp();
    if (n == 0) STAMP(8);
    n += cnt; seq_c += cnt;
    for (int u = 0; u < cnt; ++u) produce();
  }
  STAMP(9);
  if (timed_out && lane == 0 && cv.status) atomicOr(cv.status, STATUS_TIMEOUT);
  // the lanes that share a head add up their shares of its denominator
#pragma unroll
  for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      lrun[nt][0] += __shfl_xor_sync(0xffffffffu, lrun[nt][0], sh);
      lrun[nt][1] += __shfl_xor_sync(0xffffffffu, lrun[nt][1], sh);
    }
  __syncthreads();
  STAMP(2);

  // ---- merge the warps' partial states through shared memory ----
  // scratch: behind the stages when the pipeline runs across items (copies of the next item are landing in them),
  // otherwise the stages themselves, which are idle by now
  unsigned char *scratch = xpref ? smem + (size_t)NW * NSTAGE * 2 * TILEB : smem;
  constexpr int RS = D + 2;   // row stride of red_o in floats: spreads the transposed accumulators' stores over the banks (two-way
                              // conflicts left; four more bytes per row and a group of 8 heads no longer fits behind the stages)
  float2 *red_ml = reinterpret_cast<float2 *>(scratch);                           // [NW][16]
  float *red_o = reinterpret_cast<float *>(scratch + NW * 16 * sizeof(float2));   // [NW][g][RS]
  if (r0 == 0) {
#pragma unroll
    for (int nt = 0; nt < NTN; ++nt) {
      red_ml[warp * 16 + nt * 8 + cq] = make_float2(mrun[nt][0], lrun[nt][0]);
      red_ml[warp * 16 + nt * 8 + cq + 1] = make_float2(mrun[nt][1], lrun[nt][1]);
    }
    if (!G16) { red_ml[warp * 16 + 8 + cq] = make_float2(-INFINITY, 0.f); red_ml[warp * 16 + 9 + cq] = make_float2(-INFINITY, 0.f); }
  }
#pragma unroll
  for (int nt = 0; nt < NTN; ++nt) {
    const int hq = nt * 8 + cq;
#pragma unroll
    for (int t = 0; t < D / 16; ++t) {
      if (hq < g) {
        red_o[((size_t)warp * g + hq) * RS + t * 16 + r0] = oT[nt][t][0];
        red_o[((size_t)warp * g + hq) * RS + t * 16 + r0 + 8] = oT[nt][t][2];
      }
      if (hq + 1 < g) {
        red_o[((size_t)warp * g + hq + 1) * RS + t * 16 + r0] = oT[nt][t][1];
        red_o[((size_t)warp * g + hq + 1) * RS + t * 16 + r0 + 8] = oT[nt][t][3];
      }
    }
  }
  __syncthreads();
  // A head served by a single CTA is finished here (bf16 output, final max and denominator); otherwise the CTA
  // leaves one partial in global memory.  The prefill scoring pass always leaves partials.
  STAMP(20);
  const HeadItems hi{it.hd_first, it.hd_count};   // travels with the item: no load on the way to the merge
  const bool direct = hi.count == 1 && a.mode != ATTN_PREFILL;
  if (hi.count > 0) STAMP(21);
  for (int pr = threadIdx.x; pr < g * D / 2; pr += NW * 32) {
    const int idx = pr * 2, row = idx / D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) M = fmaxf(M, red_ml[w * 16 + row].x);
    float a0 = 0.f, a1 = 0.f, L = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float2 ml = red_ml[w * 16 + row];
        const float f = exp2f(ml.x - M);   // a warp without work has m = -inf -> factor 0
        const float2 x = *reinterpret_cast<const float2 *>(red_o + ((size_t)w * g + row) * RS + (idx - row * D));
        a0 += x.x * f; a1 += x.y * f;
        L += ml.y * f;
      }
    }
    if (direct) {
      const float inv = L > 0.f ? 1.f / L : 0.f;
      *reinterpret_cast<uint32_t *>(a.out + ((long long)it.i * G.Hq + (long long)it.h * g) * D + idx) = pack_bf16(a0 * inv, a1 * inv);
      if (idx % D == 0) a.head_mz[(long long)it.i * G.Hq + it.h * g + row] = make_float2(M, L);
    } else {
      *reinterpret_cast<float2 *>(a.part_o + (long long)item_idx * g * D + idx) = make_float2(a0, a1);
      if (idx % D == 0) a.part_ml[(long long)item_idx * g + row] = make_float2(M, L);
    }
  }
  STAMP(3);
  KSTAMP_MAX(kslot, 2);
  if (direct || a.mode == ATTN_PREFILL) continue;

  // ---- the CTA that finishes this head last merges its split partials ----
  // Every thread's partial stores are ordered before the barrier; thread 0's fence after it makes them visible device-wide
  // before the head's counter moves (cumulative over the barrier).  The CTA that comes last reads the partials past L1,
  // after it has seen the final count.
  __syncthreads();
  if (threadIdx.x == 0) {
    int *ctr = a.head_done + it.i * G.Hkv + it.h;
    __threadfence();
    const int prev = atomicAdd(ctr, 1);
    s_flag = prev == hi.count - 1;
    if (s_flag) *ctr = 0;
  }
  __syncthreads();
  STAMP(4);
  if (!s_flag) continue;
  STAMP(22);
  constexpr int NT = NW * 32;
  {
    // Each thread owns four output columns of one query head.  The partials of up to MB splits are fetched in one
    // batch of independent loads (one L2 round trip); longer heads continue with an online log-sum-exp merge.
#ifndef WNW_MERGE_BATCH
#define WNW_MERGE_BATCH 16
#endif
    constexpr int MB = WNW_MERGE_BATCH;
    const int nvec = g * D / 4;
    const float4 *po = reinterpret_cast<const float4 *>(a.part_o + (long long)hi.first * g * D);
    const float2 *pml = a.part_ml + (long long)hi.first * g;
    bf16 *ob = a.out + ((long long)it.i * G.Hq + (long long)it.h * g) * D;
    for (int v = threadIdx.x; v < nvec; v += NT) {
      const int row = v * 4 / D;
      float M = -INFINITY, Z = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int n0 = 0; n0 < hi.count; n0 += MB) {
        float2 ml[MB];
        float4 x[MB];
#pragma unroll
        for (int j = 0; j < MB; ++j) {
          if (n0 + j < hi.count) {
            ml[j] = __ldcg(pml + (long long)(n0 + j) * g + row);
            x[j] = __ldcg(po + (long long)(n0 + j) * nvec + v);
          } else {
            ml[j] = make_float2(-INFINITY, 0.f);
            x[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        float Mb = M;
#pragma unroll
        for (int j = 0; j < MB; ++j) Mb = fmaxf(Mb, ml[j].x);
        if (Mb > -INFINITY) {
          const float sc0 = exp2f(M - Mb);  // M = -inf on the first batch -> 0
          acc.x *= sc0; acc.y *= sc0; acc.z *= sc0; acc.w *= sc0; Z *= sc0;
#pragma unroll
          for (int j = 0; j < MB; ++j) {
            const float w = exp2f(ml[j].x - Mb);  // empty split: m = -inf -> 0
            acc.x += x[j].x * w; acc.y += x[j].y * w; acc.z += x[j].z * w; acc.w += x[j].w * w;
            Z += ml[j].y * w;
          }
          M = Mb;
        }
      }
      const float inv = Z > 0.f ? 1.f / Z : 0.f;
      uint2 packed;
      packed.x = pack_bf16(acc.x * inv, acc.y * inv);
      packed.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2 *>(ob + v * 4) = packed;
      if (v % (D / 4) == 0) a.head_mz[(long long)it.i * G.Hq + it.h * g + row] = make_float2(M, Z);
    }
  }
  STAMP(5);
  KSTAMP_MAX(kslot, 2);
  }  // work items of this CTA
  // after a timeout copies may still be in flight towards this CTA's shared memory: bounded wait before it is released
  for (; seq_c < seq_p; ++seq_c) {
    const int stage = (int)(seq_c % NSTAGE);
    if ((ring[warp][stage].x & 256) && !((prewaited >> stage) & 1u)) {
      mbar_wait(smem_u32(&bars[warp][stage]), (phase_bits >> stage) & 1u);
      phase_bits ^= 1u << stage;
    }
  }
  GSTAMP(15);
  STAMPV(27, q_end - q_begin);
  STAMPV(28, seq_c);
  pdl_finish();
}

template <int D, bool G16, int NW, int VAR>
__global__ void __launch_bounds__(NW * 32, NW == NW_THR ? (G16 ? 2 : WNW_THR_CTAS_PER_SM) : 1) wnw_attn_kernel(const __grid_constant__ CacheView cv,
                                                           const __grid_constant__ AttnArgs a,
                                                           const __grid_constant__ InlineItems inl,
                                                           const __grid_constant__ TmaMaps maps) {
  attn_body<D, G16, NW, VAR>(cv, a, &inl, maps, (int)blockIdx.x);
}

// The CTAs of several layers in one launch (layers whose inputs are all ready and whose outputs are read after the
// step): CTA x belongs to the layer whose range of the prefix table holds x and does exactly what it would do in that
// layer's own launch.
// The register cap leaves room on the SM for a recall CTA (256 threads x 40 registers) beside an 8-warp attention CTA:
// the recall of the previous step runs while this launch fills the machine.  (The layer's arguments are read through a
// run-time index into the parameters, which costs registers: uncapped this kernel takes about 240, and the recall then
// waits for attention CTAs to retire: config 1 back to back 84 us per step.)
template <int D, bool G16, int NW, int VAR>
__global__ void __maxnreg__(NW == 8 ? 208 : 255) wnw_attn_multi_kernel(const __grid_constant__ CacheView cv,
                                                                 const __grid_constant__ MultiArgs m,
                                                                 const __grid_constant__ TmaMaps maps) {
  int l = 0;
  while (l + 1 < m.n && (int)blockIdx.x >= m.cta_prefix[l + 1]) ++l;
  attn_body<D, G16, NW, VAR>(cv, m.l[l], nullptr, maps, (int)blockIdx.x - m.cta_prefix[l] + m.cta_first[l]);
}

template <int D, bool G16, int NW, int VAR>
static cudaError_t launch_multi_tb(const CacheView &cv, const MultiArgs &m, size_t smem, const TmaMaps &maps, bool pdl,
                                   cudaStream_t st) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)m.cta_prefix[m.n], 1, 1);
  cfg.blockDim = dim3(NW * 32, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, wnw_attn_multi_kernel<D, G16, NW, VAR>, cv, m, maps);
}

template <int D, bool G16, int NW, int VAR>
static cudaError_t launch_tb(const CacheView &cv, const AttnArgs &a, cudaStream_t st) {
  // stages + slack to align them to the swizzle atom + the merge scratch when it does not alias the stages
  const size_t smem = (size_t)NW * nstage_of(NW) * 2 * GR * D * 2 + 1024 + (a.xpref ? attn_scratch_bytes(NW, cv.geo.g, D) : 0);
  if (!a.maps) return cudaErrorInvalidValue;
  InlineItems inl;
  if (a.n_items <= INLINE_ITEMS_MAX && a.items_host) memcpy(inl.it, a.items_host, sizeof(WorkItem) * a.n_items);
  else if (a.n_items <= INLINE_ITEMS_MAX) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(a.cta_ranges ? a.n_ctas : a.n_items), 1, 1);
  cfg.blockDim = dim3(NW * 32, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (a.pdl) {  // let this launch begin before the previous kernel in the stream has drained (see griddepcontrol above)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, wnw_attn_kernel<D, G16, NW, VAR>, cv, a, inl, *a.maps);
}
template <int D, bool G16, int NW>
static cudaError_t launch_t(const CacheView &cv, const AttnArgs &a, cudaStream_t st) {
  if constexpr (D == 128)
    if (cv.geo.kv8) return launch_tb<D, G16, NW, 2>(cv, a, st);
  if (cv.geo.kv8) return cudaErrorInvalidValue;
  return cv.geo.token_base ? launch_tb<D, G16, NW, 1>(cv, a, st) : launch_tb<D, G16, NW, 0>(cv, a, st);
}

// ---- TMA descriptors ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn tiled_encoder() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {  // the driver entry point is looked up at run time: the library does not link against libcuda
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess || !p ||
        qres != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    fn = (EncodeTiledFn)p;
  }
  return fn;
}

bool encode_store_map(CUtensorMap *map, const void *base, unsigned long long rows, int d) {
  const EncodeTiledFn fn = tiled_encoder();
  if (!fn) return false;
  if (rows < 1) rows = 1;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};          // bytes between rows
  const cuuint32_t box[2] = {64, (cuuint32_t)GR};              // 128 bytes x 16 rows
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The slot pool of an e4m3 tidal tier: rows of 128 one-byte elements (head_dim 128), boxes of 16 rows, 128-byte swizzle.
bool encode_store_map_e4m3(CUtensorMap *map, const void *base, unsigned long long rows) {
  const EncodeTiledFn fn = tiled_encoder();
  if (!fn) return false;
  if (rows < 1) rows = 1;
  const cuuint64_t dims[2] = {128, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {128, (cuuint32_t)GR};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool G16, int NW>
static cudaError_t configure_t() {
  const size_t want = (size_t)NW * nstage_of(NW) * 2 * GR * D * 2 + 1024 + attn_scratch_bytes(NW, G16 ? 16 : 8, D);
  const int bytes = (int)std::min<size_t>(want, 227 * 1024 - 512);   // what a CTA may have, less this kernel's static shared memory
  cudaError_t e = cudaFuncSetAttribute(wnw_attn_kernel<D, G16, NW, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(wnw_attn_multi_kernel<D, G16, NW, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(wnw_attn_multi_kernel<D, G16, NW, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e;
  if constexpr (D == 128) {   // the e4m3 tidal tier
    if ((e = cudaFuncSetAttribute(wnw_attn_kernel<D, G16, NW, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(wnw_attn_multi_kernel<D, G16, NW, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e;
  }
  return cudaFuncSetAttribute(wnw_attn_kernel<D, G16, NW, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}
// Opt-in shared-memory sizes, set once per device at cache creation (never during a stream capture).
cudaError_t configure_attn_kernels() {
  cudaError_t e;
  if ((e = configure_t<128, true, NW_LAT>()) != cudaSuccess) return e;
  if ((e = configure_t<128, false, NW_LAT>()) != cudaSuccess) return e;
  if ((e = configure_t<64, true, NW_LAT>()) != cudaSuccess) return e;
  if ((e = configure_t<64, false, NW_LAT>()) != cudaSuccess) return e;
  if ((e = configure_t<128, true, NW_THR>()) != cudaSuccess) return e;
  if ((e = configure_t<128, false, NW_THR>()) != cudaSuccess) return e;
  if ((e = configure_t<64, true, NW_THR>()) != cudaSuccess) return e;
  return configure_t<64, false, NW_THR>();
}

cudaError_t launch_attn(const CacheView &cv, const AttnArgs &a, cudaStream_t st) {
  if (a.n_items <= 0) return cudaSuccess;
  const bool g16 = cv.geo.g > 8;
  if (a.throughput) {
    if (cv.geo.d == 128) return g16 ? launch_t<128, true, NW_THR>(cv, a, st) : launch_t<128, false, NW_THR>(cv, a, st);
    if (cv.geo.d == 64) return g16 ? launch_t<64, true, NW_THR>(cv, a, st) : launch_t<64, false, NW_THR>(cv, a, st);
  } else {
    if (cv.geo.d == 128) return g16 ? launch_t<128, true, NW_LAT>(cv, a, st) : launch_t<128, false, NW_LAT>(cv, a, st);
    if (cv.geo.d == 64) return g16 ? launch_t<64, true, NW_LAT>(cv, a, st) : launch_t<64, false, NW_LAT>(cv, a, st);
  }
  return cudaErrorInvalidValue;
}

// One launch for the CTAs of n layers (all cut for the one-shot 8-warp variant).
cudaError_t launch_attn_multi(const CacheView &cv, const AttnArgs *args, int n, const int *first_cta, const int *count_cta,
                              bool pdl, cudaStream_t st) {
  if (n <= 0 || n > MULTI_LAYERS_MAX || ((first_cta == nullptr) != (count_cta == nullptr))) return cudaErrorInvalidValue;
  MultiArgs m;
  memset(&m, 0, sizeof(m));
  size_t smem = 0;
  int ctas = 0, n_used = 0;
  const int d = cv.geo.d;
  for (int i = 0; i < n; ++i) {
    const AttnArgs &a = args[i];
    if (a.n_items <= 0) continue;
    if (a.throughput || !a.maps || a.maps != args[0].maps) return cudaErrorInvalidValue;
    const int all = a.cta_ranges ? a.n_ctas : a.n_items;
    const int first = first_cta ? first_cta[i] : 0, count = count_cta ? count_cta[i] : all;
    if (first < 0 || count < 0 || first + count > all) return cudaErrorInvalidValue;
    if (count == 0) continue;
    m.cta_prefix[n_used] = ctas;
    m.cta_first[n_used] = first;
    m.l[n_used] = a;
    m.l[n_used].pdl = 0; m.l[n_used].wait_inputs = 0;
    ++n_used;
    ctas += count;
    smem = std::max(smem, (size_t)NW_LAT * nstage_of(NW_LAT) * 2 * GR * d * 2 + 1024 + (a.xpref ? attn_scratch_bytes(NW_LAT, cv.geo.g, d) : 0));
  }
  if (n_used == 0) return cudaSuccess;
  m.n = n_used; m.cta_prefix[n_used] = ctas;
  const bool g16 = cv.geo.g > 8, tb = cv.geo.token_base != 0;
  const TmaMaps &maps = *args[0].maps;
  if (d == 128 && cv.geo.kv8)
    return g16 ? launch_multi_tb<128, true, NW_LAT, 2>(cv, m, smem, maps, pdl, st) : launch_multi_tb<128, false, NW_LAT, 2>(cv, m, smem, maps, pdl, st);
  if (d == 128) {
    if (g16) return tb ? launch_multi_tb<128, true, NW_LAT, 1>(cv, m, smem, maps, pdl, st) : launch_multi_tb<128, true, NW_LAT, 0>(cv, m, smem, maps, pdl, st);
    return tb ? launch_multi_tb<128, false, NW_LAT, 1>(cv, m, smem, maps, pdl, st) : launch_multi_tb<128, false, NW_LAT, 0>(cv, m, smem, maps, pdl, st);
  }
  if (d == 64 && !cv.geo.kv8) {
    if (g16) return tb ? launch_multi_tb<64, true, NW_LAT, 1>(cv, m, smem, maps, pdl, st) : launch_multi_tb<64, true, NW_LAT, 0>(cv, m, smem, maps, pdl, st);
    return tb ? launch_multi_tb<64, false, NW_LAT, 1>(cv, m, smem, maps, pdl, st) : launch_multi_tb<64, false, NW_LAT, 0>(cv, m, smem, maps, pdl, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace wnw
