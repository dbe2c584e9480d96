// wnw_attend_static: one-query full attention over a caller-owned K/V buffer, with every byte of scratch taken
// from a fixed array inside the library image.  It reuses the split-K attention kernel of wnw_attn.cu unchanged;
// what differs from the cache-based entry points is only where the split partials, the completion counters and
// the per-head split table live.
//
// Who this is for: callers that cannot allocate device memory at the point of the call.  A serving loop that has
// handed the whole device to its own pool allocator, or a latency-critical decode thread for which the implicit
// device-wide synchronisation of cudaMalloc/cudaFree is not acceptable, can still run an attention step through
// this entry point: it calls no cudaMalloc, no cudaFree and no allocating library routine, and its host side keeps
// its work list on the stack.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "../../include/wnw.h"
#include "wnw_internal.cuh"

using namespace wnw;

namespace {

constexpr int ST_MAX_KV_HEADS = 64;
constexpr int ST_MAX_Q_HEADS = 128;
constexpr int ST_MAX_ITEMS = INLINE_ITEMS_MAX;       // the item list travels in kernel parameters
constexpr long long ST_MAX_TOKENS = 1ll << 20;
constexpr int ST_MAX_DEVICES = 64;

// layout of the scratch array (byte offsets, all multiples of 256)
constexpr size_t OFF_ZERO = 0;                                                     // zero words (text length = 0)
constexpr size_t OFF_STATUS = 192;                                                 // int32: sticky STATUS_* bits of the kernels' bounded waits;
                                                                                   //   survives the per-call clearing, reset when it is read
constexpr size_t OFF_COUNTERS = 256;                                               // int32 [ST_MAX_KV_HEADS]
constexpr size_t OFF_HEAD_MZ = 1024;                                               // float2 [ST_MAX_Q_HEADS]
constexpr size_t OFF_PART_ML = 2048;                                               // float2 [ST_MAX_ITEMS][MAX_G]
constexpr size_t OFF_PART_O = OFF_PART_ML + (size_t)ST_MAX_ITEMS * MAX_G * 8;      // float  [ST_MAX_ITEMS][MAX_G][128]
constexpr size_t SCRATCH_BYTES = OFF_PART_O + (size_t)ST_MAX_ITEMS * MAX_G * 128 * 4;  // about 0.8 MB
static_assert(OFF_PART_O % 256 == 0, "scratch sections are 256-byte aligned");

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

// In host code the array's name is only a stand-in; the device address comes from cudaGetSymbolAddress, once per device.
unsigned char *g_scratch_addr[ST_MAX_DEVICES] = {nullptr};

wnw_status_t scratch_for_current_device(int device, unsigned char **out) {
  if (device < 0 || device >= ST_MAX_DEVICES) return WNW_ERR_INVALID_ARG;
  if (!g_scratch_addr[device]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return WNW_ERR_CUDA; }
    if (configure_attn_kernels() != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }  // shared-memory opt-in, no allocation
    g_scratch_addr[device] = (unsigned char *)p;
  }
  *out = g_scratch_addr[device];
  return WNW_OK;
}

// Per call, on the caller's stream ahead of the attention kernel: clears what must start at zero (the zero words, the
// heads' completion counters).  The array keeps the previous call's contents otherwise; the status word is left alone.
__global__ void static_prepare_kernel(unsigned char *scr) {
  const int t = threadIdx.x;
  if (t < (int)(OFF_STATUS / 4)) reinterpret_cast<int32_t *>(scr + OFF_ZERO)[t] = 0;
  if (t < ST_MAX_KV_HEADS) reinterpret_cast<int32_t *>(scr + OFF_COUNTERS)[t] = 0;
}

}  // namespace

extern "C" wnw_status_t wnw_attend_static_status(int32_t device, void *cuda_stream, int32_t *timed_out) {
  if (!timed_out) return WNW_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }
  if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }
  struct Restore { int prev, dev; ~Restore() { if (prev != dev) cudaSetDevice(prev); } } restore{prev, device};
  unsigned char *scr = nullptr;
  wnw_status_t rc = scratch_for_current_device(device, &scr);
  if (rc != WNW_OK) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, scr + OFF_STATUS, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(scr + OFF_STATUS, 0, sizeof(word), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return WNW_ERR_CUDA;
  }
  *timed_out = (word & STATUS_TIMEOUT) ? 1 : 0;
  return WNW_OK;
}

extern "C" wnw_status_t wnw_attend_static(const void *kv_dev, int32_t n_tokens, int32_t padded_tokens, const void *q_dev,
                                          void *out_dev, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                          float softmax_scale, int32_t device, void *cuda_stream) {
  if (!kv_dev || !q_dev || !out_dev) return WNW_ERR_INVALID_ARG;
  if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || n_tokens < 1) return WNW_ERR_INVALID_ARG;
  if (padded_tokens < n_tokens || padded_tokens % GR) return WNW_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || std::isinf(softmax_scale)) return WNW_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return WNW_ERR_UNSUPPORTED;
  // beyond the fixed scratch: refuse rather than overrun
  if (n_kv_heads > ST_MAX_KV_HEADS || n_q_heads > ST_MAX_Q_HEADS || n_q_heads / n_kv_heads > MAX_G ||
      (long long)padded_tokens > ST_MAX_TOKENS)
    return WNW_ERR_CAPACITY;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }
  if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }
  struct Restore { int prev, dev; ~Restore() { if (prev != dev) cudaSetDevice(prev); } } restore{prev, device};
  unsigned char *scr = nullptr;
  wnw_status_t rc = scratch_for_current_device(device, &scr);
  if (rc != WNW_OK) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  // split every head's granules over at most ST_MAX_ITEMS CTAs in total
  const int nw = attn_warps(false);
  const int n_gran = (n_tokens + GR - 1) / GR;
  const int per_head_max = ST_MAX_ITEMS / n_kv_heads;
  if (per_head_max < 1) return WNW_ERR_CAPACITY;
  int gpi = std::max(nw, (n_gran + per_head_max - 1) / per_head_max);
  gpi = (gpi + nw - 1) / nw * nw;
  const int n_cta = (n_gran + gpi - 1) / gpi;
  if (n_cta * n_kv_heads > ST_MAX_ITEMS) return WNW_ERR_CAPACITY;
  WorkItem items[ST_MAX_ITEMS];   // on the stack: the list travels in the kernel's parameters
  int n_items = 0;
  for (int h = 0; h < n_kv_heads; ++h)
    for (int x = 0; x < n_cta; ++x) {
      const int g0 = (int)((long long)n_gran * x / n_cta), g1 = (int)((long long)n_gran * (x + 1) / n_cta);
      items[n_items++] = WorkItem{0, h, g0, g1, 0, ROLE_ANCHOR, h, n_tokens, n_gran, 0, 0, h * n_cta, n_cta};
    }

  CacheView cv;
  memset(&cv, 0, sizeof(cv));
  Geometry &G = cv.geo;
  G.L = 1; G.Hq = n_q_heads; G.Hkv = n_kv_heads; G.d = head_dim; G.g = n_q_heads / n_kv_heads;
  G.nc = GR; G.ncp = GR; G.gpc = 1; G.topk = 0;
  G.T_cap_pad = GR; G.n_tg = 0;                        // no text region: every key comes from kv_dev
  G.C_max = padded_tokens / GR; G.S_max = 0; G.T_a_pad = padded_tokens;
  G.max_batch = 1;
  const double scale = softmax_scale > 0.f ? (double)softmax_scale : 1.0 / std::sqrt((double)head_dim);
  G.scale_log2 = (float)(scale * 1.4426950408889634);
  cv.text = reinterpret_cast<bf16 *>(scr + OFF_ZERO);
  cv.text_len = reinterpret_cast<int32_t *>(scr + OFF_ZERO);
  cv.status = reinterpret_cast<int32_t *>(scr + OFF_STATUS);   // where a bounded wait that ran out leaves its mark

  // the array keeps the previous call's contents: clear what must start at zero
  static_prepare_kernel<<<1, 64, 0, st>>>(scr);
  if (cudaGetLastError() != cudaSuccess) return WNW_ERR_CUDA;

  // descriptor of the caller's buffer (a host-side encode, no allocation); every role points at it
  TmaMaps maps;
  if (!encode_store_map(&maps.anchor, kv_dev, (unsigned long long)n_kv_heads * 2 * padded_tokens, head_dim)) return WNW_ERR_CUDA;
  maps.text = maps.pool = maps.fixed = maps.anchor;
  AttnArgs a{};
  a.maps = &maps;
  a.mode = ATTN_FULL; a.layer = 0; a.n_active = 1; a.has_new = 0; a.score_on = 0;
  a.items = nullptr; a.items_host = items; a.n_items = n_items; a.pdl = 0;
  a.q = (const bf16 *)q_dev;
  a.anchor_base = (const bf16 *)kv_dev; a.anchor_seq_stride = 0; a.anchor_head0 = 0;
  a.part_o = reinterpret_cast<float *>(scr + OFF_PART_O);
  a.part_ml = reinterpret_cast<float2 *>(scr + OFF_PART_ML);
  a.gran_em = nullptr; a.n_aq = 1; a.n_ag_max = 1;
  a.head_done = reinterpret_cast<int32_t *>(scr + OFF_COUNTERS);
  a.head_mz = reinterpret_cast<float2 *>(scr + OFF_HEAD_MZ);
  a.out = (bf16 *)out_dev;
  if (launch_attn(cv, a, st) != cudaSuccess) { cudaGetLastError(); return WNW_ERR_CUDA; }
  return WNW_OK;
}
