/*
 * WnW decode-step ORACLE -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow CPU restatement of the decode-time hot path of the
 * Waxing-and-Waning KV cache (Method section: "Method Overview", "Prefill
 * Compression", "Decode-Step Score Aggregation" (Eq. 2), "Dynamic Chunk
 * Selection"), in the chunk-granular, hard-budget, per-layer form this
 * repository builds.  Only tests, the smoke check and the benchmark's CPU
 * baseline leg may call it.  It shares no code with the CUDA library.
 *
 * How it differs in structure from the CUDA path, on purpose:
 *   - it keeps the FULL, never-moved K and V of every head (also what fixed
 *     heads discard and what tidal heads offload); there is no slot pool, no
 *     host mirror and no copy;
 *   - residency is a table of chunk ids; attention is a masked softmax over the
 *     full key set, accumulated in double precision;
 *   - every table update of a step happens in wnwo_step_end, after all layers
 *     (the paper's order: "after attention is computed for all L layers").
 *
 * Pins (tests/, CPU only): softmax rows sum to one; budget 1.0 equals a dense
 * softmax attention written separately with numpy; chunk scores sum to the
 * anchor heads' audio attention mass; closed forms for identical keys and for a
 * one-hot key; top-k against brute force; the table update against an
 * independent set model and a hand-worked trace.  The numeric trajectory on
 * seeded inputs has no printed example in the paper: beyond those invariants
 * it is "parity unpinned".
 *
 * Conventions (all chosen readings are listed in the design document):
 *   - inputs are bf16 bit patterns (uint16); all arithmetic is double;
 *   - softmax runs over the head's whole allowed key set, text and audio
 *     (Eq. 2 takes the audio entries of that softmax);
 *   - score_sum[c] = sum over the layer's anchor q-heads and over tau in chunk
 *     c of the softmax weight; the ranking key is the chunk MEAN,
 *     (float)score_sum[c] / (float)len_c, compared as float, ties to the lower
 *     chunk index;
 *   - score scope PER_LAYER: a layer without anchor heads ranks by the scores
 *     of the nearest layer that has one (ties to the lower layer); score scope
 *     GLOBAL (Eq. 2 as printed): every tidal layer ranks by the sum of the
 *     scores of ALL anchor layers of the step, added in layer order;
 *   - a selection made at step s is used by tidal attention at step s+1;
 *   - slots S = max(1, floor((double)budget * C + 1e-6)), capped at C;
 *   - stamps: a chunk selected with rank r at step s gets s*topk + (topk-1-r);
 *     prefill gives rank r the stamp -1-r;
 *   - residency SEGMENT_LAG (Chunk Structure + Dynamic Chunk Selection as printed):
 *     the storage unit (`chunk` tokens) is a SEGMENT; a chunk is two consecutive
 *     segments, so adjacent chunks share one; chunk j = segments {j, j+1}, ranked
 *     by the mean over its tokens, (float)(sum_j + sum_{j+1}) / (len_j + len_{j+1});
 *     the segments placed at prefill stay resident for good (slots [0, S_base));
 *     the segments of the selected chunks that are not resident are fetched into
 *     dynamic slots [S_base, S); a fetched segment left unselected for delta
 *     consecutive steps is dropped (its stamp = the step it was last selected in).
 *     D = S - S_base = 2*topk*(delta+1) dynamic slots always suffice.
 *   - token-granular prefill compression of FIXED heads (wnwo_place_prefill_tokens; "Prefill Compression" as
 *     printed, Eq. 1 for the per-head retention): p_prefill[tau] = sum over the text queries and the head's q-heads
 *     of the softmax weight of tau; the ranking key is (float)p_prefill[tau], ties to the earlier position; every
 *     segment of `seg` tokens keeps its floor((double)retention * length) best positions (variant 1: the same total
 *     from the whole head); the head then attends to [text | kept positions].  Tidal tables stay chunk-granular,
 *     except with residency 2 (SEGMENT_LAG with a token-granular base): no segment is permanent as a whole; every tidal
 *     head keeps its own best positions for good (either variant) and attends to [text | its kept
 *     positions | all positions of the segments resident in the layer's dynamic slots]; a selected segment that is
 *     not in a dynamic slot counts as a miss (its complement has to be fetched).
 *     Pinned in tests/test_oracle_tokens.py against numpy sorts, a separate numpy softmax and hand-worked cases.
 *   - streaming audio (wnwo_append_audio; the Limitations section names streaming as the method's setting, the Method
 *     section does not say how a growing clip enters the tiers, so this is a reading): new audio positions extend the
 *     clip; the short last chunk fills up first, then new chunks begin.  Anchor heads see every new position at once.
 *     Tidal heads see a new position only through the residency table: new positions of a chunk that is resident are
 *     visible with it, a new chunk is on the host until the anchor heads' scores select it; the slot count follows the
 *     budget, S = max(1, floor(budget * C)) of the grown C, and the added slots start empty.  Fixed heads keep the
 *     subset chosen at prefill, which is final (Method Overview: static subset, the rest is discarded): they never see
 *     a position that arrived later, not even inside a chunk they keep.  Hard budget only.
 *     Pinned in tests/test_oracle_streaming.py: appending in pieces equals placing the whole clip (anchor heads: exactly;
 *     the full sets of every role against numpy attention over an explicit position mask), slot rule, table carry-over.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define WNWO_OK 0
#define WNWO_ERR_ARG 1
#define WNWO_ERR_STATE 2
#define WNWO_ERR_OOM 3

#define ROLE_ANCHOR 0
#define ROLE_TIDAL 1
#define ROLE_FIXED 2

typedef struct {
  int placed_layers;   /* how many layers have been placed */
  int T_a, T_t, T_cap; /* audio tokens, current text tokens, text capacity */
  int T_a_fixed;       /* audio tokens that had arrived when the sequence was placed: all a fixed head can ever see */
  int C, S;            /* chunks (segments in SEGMENT_LAG), slots of the tidal table */
  int S_base;          /* slots filled at prefill; = S with the hard budget; fixed heads keep S_base chunks */
  long long steps;     /* decode steps this sequence took part in */
  uint16_t **audK, **audV; /* [L] -> [Hkv][T_a][d]   full audio K,V of every head */
  uint16_t **txtK, **txtV; /* [L] -> [Hkv][T_cap][d] */
  int *slot_chunk;         /* [L][S]  -1 = free */
  long long *stamp;        /* [L][S] */
  int *fixed_set;          /* [L][Hkv][S] */
  int *fixed_n;            /* [L][Hkv] */
  unsigned char **tok_mask; /* [L][Hkv] -> [T_a] kept positions of a fixed head placed token by token; NULL = chunk form */
  double **tok_score;       /* [L][Hkv] -> [T_a] p_prefill of every audio position (token placement only) */
  double *score_sum;       /* [L][C]  this step's scores (anchor layers) */
  double *pre;             /* [L][Hkv][C] prefill scores */
  int *sel;                /* [L][topk] */
  int *n_sel;              /* [L] */
  long long hits, misses, evictions;
} Seq;

typedef struct {
  int L, Hq, Hkv, d, g, chunk, topk, max_batch, max_audio, max_text;
  int scope;      /* 0: per layer with nearest-anchor routing; 1: global sum over all anchor layers */
  int residency;  /* 0: hard budget (fixed pool, least-recently-selected eviction); 1: SEGMENT_LAG; 2: SEGMENT_LAG with a
                     token-granular permanent base (tidal heads keep their best positions of every segment) */
  int delta;      /* eviction lag of SEGMENT_LAG */
  double budget, scale;
  uint8_t *roles; /* [L][Hkv] */
  uint8_t *anchor_layer; /* [L] does the layer have an anchor head: over ALL KV heads of the model, which are more than this
                          * oracle's own when it holds one shard of the heads (wnwo_create_shard) */
  int sharded;    /* this oracle holds a shard of the KV heads: its chunk scores are partial sums until the shards' sums have
                   * been added up and handed back (wnwo_set_chunk_scores) */
  int *src;       /* [L] score source layer, -1 if the layer has no tidal heads or no source */
  Seq *seq;
  int *active;
  int n_active;
  int in_step, next_layer, appended;
} Oracle;

static double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

static int layer_has(const Oracle *o, int l, int role) {
  for (int h = 0; h < o->Hkv; ++h)
    if (o->roles[l * o->Hkv + h] == role) return 1;
  return 0;
}

static int chunk_len(const Oracle *o, const Seq *s, int c) {
  int lo = c * o->chunk, hi = lo + o->chunk;
  if (hi > s->T_a) hi = s->T_a;
  return hi - lo;
}

/* ------------------------------------------------------------------ */
/* Pure pieces, exported so tests can drive them on arbitrary arrays.   */
/* ------------------------------------------------------------------ */

/* Dynamic Chunk Selection: rank chunks by mean score, (key desc, index asc).
 * score_sum as float; lens = tokens per chunk.  Writes the first k ranks. */
int wnwo_topk(const float *score_sum, const int *lens, int C, int k, int *sel_out) {
  if (k > C) k = C;
  unsigned char *taken = (unsigned char *)calloc((size_t)(C > 0 ? C : 1), 1);
  if (!taken) return -1;
  for (int r = 0; r < k; ++r) {
    int best = -1;
    float best_key = 0.f;
    for (int c = 0; c < C; ++c) {
      if (taken[c]) continue;
      float key = score_sum[c] / (float)lens[c];
      if (best < 0 || key > best_key) { /* strict > keeps the lower index on ties */
        best = c;
        best_key = key;
      }
    }
    taken[best] = 1;
    sel_out[r] = best;
  }
  free(taken);
  return k;
}

/* Chunk swap under a fixed slot pool.  sel in rank order.  Updates the table in
 * place; plan_chunk/plan_slot receive the misses (chunks to recall and where),
 * evicted[] the chunk that was displaced or -1.  Returns the number of misses. */
int wnwo_table_update(int *slot_chunk, long long *stamp, int S, const int *sel, int k, long long step, int topk,
                      int *plan_chunk, int *plan_slot, int *evicted, int *n_hits) {
  int n_plan = 0, hits = 0;
  for (int r = 0; r < k; ++r) {
    int c = sel[r];
    long long st = step * (long long)topk + (long long)(topk - 1 - r);
    int j = -1;
    for (int i = 0; i < S; ++i)
      if (slot_chunk[i] == c) j = i;
    if (j >= 0) { /* hit: refresh recency */
      stamp[j] = st;
      ++hits;
      continue;
    }
    for (int i = 0; i < S && j < 0; ++i)
      if (slot_chunk[i] < 0) j = i; /* lowest-index free slot */
    int victim = -1;
    if (j < 0) { /* least recently selected resident that is not selected now */
      for (int i = 0; i < S; ++i) {
        int in_sel = 0;
        for (int q = 0; q < k; ++q)
          if (sel[q] == slot_chunk[i]) in_sel = 1;
        if (in_sel) continue;
        if (j < 0 || stamp[i] < stamp[j]) j = i;
      }
      if (j < 0) return -1; /* cannot happen when S >= k */
      victim = slot_chunk[j];
    }
    slot_chunk[j] = c;
    stamp[j] = st;
    plan_chunk[n_plan] = c;
    plan_slot[n_plan] = j;
    evicted[n_plan] = victim;
    ++n_plan;
  }
  if (n_hits) *n_hits = hits;
  return n_plan;
}

/* Dynamic Chunk Selection over OVERLAPPING chunks (Chunk Structure): chunk j is segments j and j+1 (a clip of one
 * segment has the single chunk {0}).  seg_sum as float, lens = tokens per segment.  Writes the k best chunks in rank
 * order to sel_chunks and their segments, in that order without repeats, to segs; returns the number of segments. */
int wnwo_select_segments(const float *seg_sum, const int *lens, int n_seg, int k, int *sel_chunks, int *n_sel, int *segs) {
  const int n_ch = n_seg > 1 ? n_seg - 1 : n_seg;
  if (k > n_ch) k = n_ch;
  float *ch_sum = (float *)malloc(sizeof(float) * (size_t)(n_ch > 0 ? n_ch : 1));
  int *ch_len = (int *)malloc(sizeof(int) * (size_t)(n_ch > 0 ? n_ch : 1));
  if (!ch_sum || !ch_len) { free(ch_sum); free(ch_len); return -1; }
  for (int j = 0; j < n_ch; ++j) {
    ch_sum[j] = n_seg > 1 ? seg_sum[j] + seg_sum[j + 1] : seg_sum[j]; /* float add: the decision precision */
    ch_len[j] = n_seg > 1 ? lens[j] + lens[j + 1] : lens[j];
  }
  k = wnwo_topk(ch_sum, ch_len, n_ch, k, sel_chunks);
  free(ch_sum); free(ch_len);
  if (k < 0) return -1;
  int n = 0;
  for (int r = 0; r < k; ++r)
    for (int e = 0; e < (n_seg > 1 ? 2 : 1); ++e) {
      int g = sel_chunks[r] + e, seen = 0;
      for (int i = 0; i < n; ++i) seen |= segs[i] == g;
      if (!seen) segs[n++] = g;
    }
  if (n_sel) *n_sel = k;
  return n;
}

/* Chunk swap with a permanent base and lag-delta release (Dynamic Chunk Selection).  Slots [0, S_base) never change.
 * segs: the selected segments of this step, in order.  A selected segment that is resident is a hit (a dynamic one gets
 * stamp = step); then every dynamic slot whose segment was not selected now and has step - stamp >= delta is released;
 * then the misses take the lowest free dynamic slots in order.  released[] receives the dropped segments.
 * Returns the number of misses (plan entries), -1 if no free slot was left (cannot happen when S - S_base >= 2k(delta+1)). */
int wnwo_lag_update(int *slot_seg, long long *stamp, int S_base, int S, const int *segs, int n, long long step, int delta,
                    int *plan_seg, int *plan_slot, int *released, int *n_released, int *n_hits) {
  int hits = 0, n_rel = 0, n_plan = 0;
  unsigned char *miss = (unsigned char *)calloc((size_t)(n > 0 ? n : 1), 1);
  if (!miss) return -1;
  for (int i = 0; i < n; ++i) {
    int j = -1;
    for (int x = 0; x < S; ++x)
      if (slot_seg[x] == segs[i]) j = x;
    if (j < 0) { miss[i] = 1; continue; }
    ++hits;
    if (j >= S_base) stamp[j] = step;
  }
  for (int x = S_base; x < S; ++x) {
    if (slot_seg[x] < 0 || stamp[x] == step) continue; /* free, or selected in this step */
    if (step - stamp[x] >= (long long)delta) {
      released[n_rel++] = slot_seg[x];
      slot_seg[x] = -1;
    }
  }
  for (int i = 0; i < n; ++i) {
    if (!miss[i]) continue;
    int j = -1;
    for (int x = S_base; x < S && j < 0; ++x)
      if (slot_seg[x] < 0) j = x;
    if (j < 0) { free(miss); return -1; }
    slot_seg[j] = segs[i];
    stamp[j] = step;
    plan_seg[n_plan] = segs[i];
    plan_slot[n_plan] = j;
    ++n_plan;
  }
  free(miss);
  if (n_released) *n_released = n_rel;
  if (n_hits) *n_hits = hits;
  return n_plan;
}

/* ------------------------------------------------------------------ */
/* Life cycle                                                           */
/* ------------------------------------------------------------------ */

static void free_seq(Oracle *o, Seq *s) {
  if (s->audK)
    for (int l = 0; l < o->L; ++l) { free(s->audK[l]); free(s->audV[l]); free(s->txtK[l]); free(s->txtV[l]); }
  free(s->audK); free(s->audV); free(s->txtK); free(s->txtV);
  if (s->tok_mask) for (int i = 0; i < o->L * o->Hkv; ++i) free(s->tok_mask[i]);
  if (s->tok_score) for (int i = 0; i < o->L * o->Hkv; ++i) free(s->tok_score[i]);
  free(s->tok_mask); free(s->tok_score);
  free(s->slot_chunk); free(s->stamp); free(s->fixed_set); free(s->fixed_n);
  free(s->score_sum); free(s->pre); free(s->sel); free(s->n_sel);
  memset(s, 0, sizeof(*s));
}

void wnwo_destroy(Oracle *o) {
  if (!o) return;
  if (o->seq)
    for (int b = 0; b < o->max_batch; ++b) free_seq(o, &o->seq[b]);
  free(o->seq); free(o->roles); free(o->anchor_layer); free(o->src); free(o->active);
  free(o);
}

/* One shard of the KV heads of a model whose layers' anchor heads may sit in other shards (head-sharded serving: the only
 * thing that crosses heads is Eq. 2's chunk-score vector).  roles: this shard's heads; global_anchor_layers[l] != 0 iff layer
 * l has an anchor head in ANY shard (NULL: this oracle holds all heads).  Routing follows the global flags; a layer's
 * scores are summed over the shard's own anchor heads and are complete only after wnwo_set_chunk_scores. */
int wnwo_create_shard(int L, int Hq, int Hkv, int d, int max_batch, int max_audio, int max_text, int chunk, int topk,
                      double budget, double scale, const uint8_t *roles, int scope, int residency, int delta,
                      const uint8_t *global_anchor_layers, Oracle **out);
int wnwo_create(int L, int Hq, int Hkv, int d, int max_batch, int max_audio, int max_text, int chunk, int topk,
                double budget, double scale, const uint8_t *roles, int scope, int residency, int delta, Oracle **out) {
  return wnwo_create_shard(L, Hq, Hkv, d, max_batch, max_audio, max_text, chunk, topk, budget, scale, roles, scope, residency, delta,
                           NULL, out);
}
int wnwo_create_shard(int L, int Hq, int Hkv, int d, int max_batch, int max_audio, int max_text, int chunk, int topk,
                      double budget, double scale, const uint8_t *roles, int scope, int residency, int delta,
                      const uint8_t *global_anchor_layers, Oracle **out) {
  if (!out || !roles || L < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || d < 1 || max_batch < 1 || chunk < 1 || topk < 1)
    return WNWO_ERR_ARG;
  if (!(budget > 0.0 && budget <= 1.0) || scope < 0 || scope > 1 || residency < 0 || residency > 2 || delta < 0)
    return WNWO_ERR_ARG;
  Oracle *o = (Oracle *)calloc(1, sizeof(Oracle));
  if (!o) return WNWO_ERR_OOM;
  o->L = L; o->Hq = Hq; o->Hkv = Hkv; o->d = d; o->g = Hq / Hkv; o->chunk = chunk; o->topk = topk;
  o->max_batch = max_batch; o->max_audio = max_audio; o->max_text = max_text;
  o->budget = budget;
  o->scope = scope;
  o->residency = residency;
  o->delta = delta;
  o->scale = scale > 0.0 ? scale : 1.0 / sqrt((double)d); /* Eq. 2: q K^T / sqrt(d) */
  o->roles = (uint8_t *)malloc((size_t)L * Hkv);
  o->anchor_layer = (uint8_t *)calloc((size_t)L, 1);
  o->sharded = global_anchor_layers != NULL;
  o->src = (int *)malloc(sizeof(int) * L);
  o->seq = (Seq *)calloc((size_t)max_batch, sizeof(Seq));
  o->active = (int *)calloc((size_t)max_batch, sizeof(int));
  if (!o->roles || !o->anchor_layer || !o->src || !o->seq || !o->active) { wnwo_destroy(o); return WNWO_ERR_OOM; }
  memcpy(o->roles, roles, (size_t)L * Hkv);
  int any_anchor = 0, any_tidal = 0;
  for (int i = 0; i < L * Hkv; ++i) {
    if (roles[i] > ROLE_FIXED) { wnwo_destroy(o); return WNWO_ERR_ARG; }
    any_anchor |= roles[i] == ROLE_ANCHOR;
    any_tidal |= roles[i] == ROLE_TIDAL;
  }
  for (int l = 0; l < L; ++l) {
    o->anchor_layer[l] = global_anchor_layers ? (global_anchor_layers[l] != 0) : (uint8_t)layer_has(o, l, ROLE_ANCHOR);
    if (global_anchor_layers && layer_has(o, l, ROLE_ANCHOR) && !global_anchor_layers[l]) { wnwo_destroy(o); return WNWO_ERR_ARG; }
    any_anchor |= o->anchor_layer[l];
  }
  if (any_tidal && !any_anchor) { wnwo_destroy(o); return WNWO_ERR_ARG; }
  /* score routing: own layer if it has an anchor, else the nearest anchor layer, ties to the lower one */
  for (int l = 0; l < L; ++l) {
    o->src[l] = -1;
    if (!layer_has(o, l, ROLE_TIDAL)) continue;
    int best = -1;
    for (int a = 0; a < L; ++a) {
      if (!o->anchor_layer[a]) continue;
      if (best < 0 || abs(a - l) < abs(best - l)) best = a; /* ascending a: the lower layer wins a tie */
    }
    o->src[l] = best;
  }
  *out = o;
  return WNWO_OK;
}

int wnwo_score_source(const Oracle *o, int layer) { return (layer >= 0 && layer < o->L) ? o->src[layer] : -2; }

static int alloc_seq(Oracle *o, Seq *s, int T_a, int T_t) {
  int L = o->L, Hkv = o->Hkv, d = o->d;
  s->T_a = T_a; s->T_t = T_t; s->T_cap = o->max_text;
  s->T_a_fixed = T_a;
  s->C = (T_a + o->chunk - 1) / o->chunk;
  int S = (int)floor(o->budget * (double)s->C + 1e-6);
  if (S < 1) S = 1;
  if (S > s->C) S = s->C;
  if (o->residency == 2) S = 0; /* no whole segment is permanent: the base is a set of positions per head */
  s->S_base = S;
  if (o->residency >= 1) { /* dynamic slots for everything selected within the last delta+1 steps */
    int D = 2 * o->topk * (o->delta + 1);
    if (D > s->C - S) D = s->C - S;
    S += D;
  }
  s->S = S;
  size_t nS = (size_t)(S > 0 ? S : 1), nC = (size_t)(s->C > 0 ? s->C : 1);
  s->audK = (uint16_t **)calloc((size_t)L, sizeof(void *)); s->audV = (uint16_t **)calloc((size_t)L, sizeof(void *));
  s->txtK = (uint16_t **)calloc((size_t)L, sizeof(void *)); s->txtV = (uint16_t **)calloc((size_t)L, sizeof(void *));
  s->slot_chunk = (int *)malloc(sizeof(int) * L * nS);
  s->stamp = (long long *)calloc((size_t)L * nS, sizeof(long long));
  s->fixed_set = (int *)malloc(sizeof(int) * L * Hkv * nS);
  s->fixed_n = (int *)calloc((size_t)L * Hkv, sizeof(int));
  s->tok_mask = (unsigned char **)calloc((size_t)L * Hkv, sizeof(void *));
  s->tok_score = (double **)calloc((size_t)L * Hkv, sizeof(void *));
  s->score_sum = (double *)calloc((size_t)L * nC, sizeof(double));
  s->pre = (double *)calloc((size_t)L * Hkv * nC, sizeof(double));
  s->sel = (int *)malloc(sizeof(int) * L * o->topk);
  s->n_sel = (int *)calloc((size_t)L, sizeof(int));
  if (!s->audK || !s->audV || !s->txtK || !s->txtV || !s->slot_chunk || !s->stamp || !s->fixed_set || !s->fixed_n ||
      !s->tok_mask || !s->tok_score ||
      !s->score_sum || !s->pre || !s->sel || !s->n_sel)
    return WNWO_ERR_OOM;
  for (size_t i = 0; i < (size_t)L * nS; ++i) s->slot_chunk[i] = -1;
  for (size_t i = 0; i < (size_t)L * Hkv * nS; ++i) s->fixed_set[i] = -1;
  for (int i = 0; i < L * o->topk; ++i) s->sel[i] = -1;
  for (int l = 0; l < L; ++l) {
    size_t na = (size_t)Hkv * (size_t)(T_a > 0 ? T_a : 1) * d, nt = (size_t)Hkv * (size_t)(s->T_cap > 0 ? s->T_cap : 1) * d;
    s->audK[l] = (uint16_t *)calloc(na, 2); s->audV[l] = (uint16_t *)calloc(na, 2);
    s->txtK[l] = (uint16_t *)calloc(nt, 2); s->txtV[l] = (uint16_t *)calloc(nt, 2);
    if (!s->audK[l] || !s->audV[l] || !s->txtK[l] || !s->txtV[l]) return WNWO_ERR_OOM;
  }
  return WNWO_OK;
}

/* ------------------------------------------------------------------ */
/* Attention of one query head over an allowed key set                  */
/* ------------------------------------------------------------------ */

/* allowed[c] != 0: chunk c's audio positions are visible.  All T_t text positions
 * always are.  Writes out[d]; if chunk_mass != NULL adds the softmax weight of
 * every audio position into chunk_mass[chunk of tau]; if p_row != NULL writes
 * the whole probability row [T_t + T_a] (text first), zeros where masked. */
static void attend(const Oracle *o, const Seq *s, int layer, int kvh, const uint16_t *q, int T_t,
                   const unsigned char *allowed, double *out, double *chunk_mass, double *p_row) {
  /* a fixed head placed token by token sees exactly its kept positions; a tidal head with a token-granular base sees
   * its kept positions and every position of the segments resident in its layer's dynamic slots */
  const unsigned char *tok = s->tok_mask ? s->tok_mask[layer * o->Hkv + kvh] : NULL;
  const int tidal_base = o->roles[layer * o->Hkv + kvh] == ROLE_TIDAL;
  const int fixed_head = o->roles[layer * o->Hkv + kvh] == ROLE_FIXED;   /* sees nothing that arrived after its placement */
  const int d = o->d, T_a = s->T_a;
  const uint16_t *tK = s->txtK[layer] + (size_t)kvh * s->T_cap * d, *tV = s->txtV[layer] + (size_t)kvh * s->T_cap * d;
  const uint16_t *aK = s->audK[layer] + (size_t)kvh * T_a * d, *aV = s->audV[layer] + (size_t)kvh * T_a * d;
  const int n = T_t + T_a;
  double *logit = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
  double mx = -INFINITY;
  for (int i = 0; i < n; ++i) {
    const uint16_t *krow;
    int vis;
    if (i < T_t) { krow = tK + (size_t)i * d; vis = 1; }
    else {
      int tau = i - T_t; krow = aK + (size_t)tau * d;
      vis = tok ? (tok[tau] != 0 || (tidal_base && allowed[tau / o->chunk] != 0)) : allowed[tau / o->chunk] != 0;
      if (fixed_head && tau >= s->T_a_fixed) vis = 0;
    }
    if (!vis) { logit[i] = -INFINITY; continue; }
    double acc = 0.0;
    for (int x = 0; x < d; ++x) acc += bf16_to_double(q[x]) * bf16_to_double(krow[x]);
    logit[i] = acc * o->scale;
    if (logit[i] > mx) mx = logit[i];
  }
  for (int x = 0; x < d; ++x) out[x] = 0.0;
  if (p_row) for (int i = 0; i < n; ++i) p_row[i] = 0.0;
  if (mx == -INFINITY) { free(logit); return; } /* empty key set: zero output */
  double Z = 0.0;
  for (int i = 0; i < n; ++i)
    if (logit[i] != -INFINITY) Z += exp(logit[i] - mx);
  for (int i = 0; i < n; ++i) {
    if (logit[i] == -INFINITY) continue;
    double p = exp(logit[i] - mx) / Z;
    const uint16_t *vrow = (i < T_t) ? tV + (size_t)i * d : aV + (size_t)(i - T_t) * d;
    for (int x = 0; x < d; ++x) out[x] += p * bf16_to_double(vrow[x]);
    if (chunk_mass && i >= T_t) chunk_mass[(i - T_t) / o->chunk] += p;
    if (p_row) p_row[i] = p;
  }
  free(logit);
}

static void allowed_for(const Oracle *o, const Seq *s, int layer, int kvh, unsigned char *allowed) {
  int role = o->roles[layer * o->Hkv + kvh];
  memset(allowed, 0, (size_t)(s->C > 0 ? s->C : 1));
  if (role == ROLE_ANCHOR) {
    for (int c = 0; c < s->C; ++c) allowed[c] = 1;
  } else if (role == ROLE_TIDAL) {
    for (int j = 0; j < s->S; ++j) {
      int c = s->slot_chunk[(size_t)layer * s->S + j];
      if (c >= 0) allowed[c] = 1;
    }
  } else {
    const int *F = s->fixed_set + ((size_t)layer * o->Hkv + kvh) * s->S;
    for (int j = 0; j < s->fixed_n[layer * o->Hkv + kvh]; ++j) allowed[F[j]] = 1;
  }
}

/* ------------------------------------------------------------------ */
/* Prefill placement (Prefill Compression, restated at chunk level)     */
/* ------------------------------------------------------------------ */

/* k,v: [n_tokens][Hkv][d] bf16 bits; audio = [audio_begin, audio_end); q_last: [Hq][d]. */
/* q_text: [n_q][Hq][d], the text queries whose attention over the audio is aggregated ("Prefill Compression":
 * p_prefill = sum over text queries of their attention weights); n_q = 1 with the last prefix query is the contract's form. */
static int place_multi(Oracle *o, int seq, int layer, const uint16_t *k, const uint16_t *v, int n_tokens,
                       int audio_begin, int audio_end, const uint16_t *q_last, int n_q) {
  if (!o || seq < 0 || seq >= o->max_batch || layer < 0 || layer >= o->L || !k || !v || n_tokens < 0) return WNWO_ERR_ARG;
  if (audio_begin < 0 || audio_end < audio_begin || audio_end > n_tokens || n_q < 1) return WNWO_ERR_ARG;
  const int T_a = audio_end - audio_begin, T_t = n_tokens - T_a, Hkv = o->Hkv, d = o->d;
  if (T_a > o->max_audio || T_t > o->max_text) return WNWO_ERR_ARG;
  Seq *s = &o->seq[seq];
  if (layer == 0 && s->placed_layers != 0) { free_seq(o, s); }
  if (s->placed_layers == 0) {
    if (layer != 0) return WNWO_ERR_STATE;
    int rc = alloc_seq(o, s, T_a, T_t);
    if (rc) return rc;
  } else if (layer != s->placed_layers || T_a != s->T_a || T_t != s->T_t) {
    return WNWO_ERR_STATE;
  }
  /* copy: text positions keep their order, audio positions keep theirs */
  int ti = 0;
  for (int i = 0; i < n_tokens; ++i) {
    int is_audio = i >= audio_begin && i < audio_end;
    for (int h = 0; h < Hkv; ++h) {
      const uint16_t *ks = k + ((size_t)i * Hkv + h) * d, *vs = v + ((size_t)i * Hkv + h) * d;
      uint16_t *kd, *vd;
      if (is_audio) {
        size_t off = ((size_t)h * T_a + (size_t)(i - audio_begin)) * d;
        kd = s->audK[layer] + off; vd = s->audV[layer] + off;
      } else {
        size_t off = ((size_t)h * s->T_cap + (size_t)ti) * d;
        kd = s->txtK[layer] + off; vd = s->txtV[layer] + off;
      }
      memcpy(kd, ks, (size_t)d * 2); memcpy(vd, vs, (size_t)d * 2);
    }
    if (!is_audio) ++ti;
  }
  s->placed_layers = layer + 1;
  const int C = s->C, S = s->S;
  if (C == 0) return WNWO_OK;
  if (!q_last) return WNWO_ERR_ARG;
  /* per non-anchor KV-head: pre[c] = sum over its q-heads and tau in c of softmax(q_last K / sqrt d) over text+audio */
  unsigned char *all = (unsigned char *)malloc((size_t)C);
  double *out = (double *)malloc(sizeof(double) * d);
  int *lens = (int *)malloc(sizeof(int) * C);
  float *keyf = (float *)malloc(sizeof(float) * C);
  double *tid = (double *)calloc((size_t)C, sizeof(double));
  memset(all, 1, (size_t)C);
  for (int c = 0; c < C; ++c) lens[c] = chunk_len(o, s, c);
  int n_tid = 0;
  for (int h = 0; h < Hkv; ++h) {
    double *pre = s->pre + ((size_t)layer * Hkv + h) * C;
    for (int c = 0; c < C; ++c) pre[c] = 0.0;
    int role = o->roles[layer * Hkv + h];
    if (role == ROLE_ANCHOR) continue;
    for (int qi = 0; qi < n_q; ++qi) /* summed over the text queries, query by query, q-heads in order */
      for (int j = 0; j < o->g; ++j)
        attend(o, s, layer, h, q_last + ((size_t)qi * o->Hq + (size_t)(h * o->g + j)) * d, T_t, all, out, pre, NULL);
    if (role == ROLE_FIXED) { /* its own top-S chunks, frozen */
      for (int c = 0; c < C; ++c) keyf[c] = (float)pre[c];
      int *F = s->fixed_set + ((size_t)layer * Hkv + h) * S;
      s->fixed_n[layer * Hkv + h] = wnwo_topk(keyf, lens, C, s->S_base, F);
    } else {
      for (int c = 0; c < C; ++c) tid[c] += pre[c]; /* summed in head order */
      ++n_tid;
    }
  }
  if (n_tid > 0) { /* one table for the layer's tidal heads: rank r -> slot r, stamp -1-r */
    for (int c = 0; c < C; ++c) keyf[c] = (float)tid[c];
    int *tmp = (int *)malloc(sizeof(int) * S);
    int n = wnwo_topk(keyf, lens, C, s->S_base, tmp);
    for (int r = 0; r < n; ++r) {
      s->slot_chunk[(size_t)layer * S + r] = tmp[r];
      s->stamp[(size_t)layer * S + r] = -1 - (long long)r;
    }
    free(tmp);
  }
  free(all); free(out); free(lens); free(keyf); free(tid);
  return WNWO_OK;
}

int wnwo_place_prefill_multi(Oracle *o, int seq, int layer, const uint16_t *k, const uint16_t *v, int n_tokens,
                             int audio_begin, int audio_end, const uint16_t *q_last, int n_q) {
  if (o && o->residency == 2) return WNWO_ERR_STATE; /* a token-granular base is placed by wnwo_place_prefill_tokens */
  return place_multi(o, seq, layer, k, v, n_tokens, audio_begin, audio_end, q_last, n_q);
}

/* Eq. 1: the fraction of audio positions a tidal or fixed head keeps on the GPU, from its normalised importance
 * s_tilde in [0,1] and the scale lambda. */
void wnwo_retention_schedule(const double *s_tilde, int n, double lambda, double *retention) {
  for (int i = 0; i < n; ++i) {
    double r = s_tilde[i] * lambda;
    retention[i] = r < 1.0 ? r : 1.0;
  }
}

/* Positions a fixed head keeps ("Prefill Compression"): key[tau] = p_prefill of position tau.
 * variant 0: inside every segment of seg tokens (the last one may be shorter) the floor(retention * length) positions
 *            with the largest key; variant 1 (the ablation's global top-k): the same total number of positions, taken
 *            from the whole head with no per-segment quota.  Equal keys: the earlier position first.
 * kept: ascending positions; returns their number, or a negated error code. */
int wnwo_select_tokens(const float *key, int T_a, int seg, float retention, int variant, int *kept) {
  if (!key || !kept || T_a < 0 || seg < 1 || !(retention >= 0.0f && retention <= 1.0f)) return -WNWO_ERR_ARG;
  unsigned char *keep = (unsigned char *)calloc((size_t)(T_a > 0 ? T_a : 1), 1);
  if (!keep) return -WNWO_ERR_OOM;
  int total = 0;
  for (int lo = 0; lo < T_a; lo += seg) {
    int len = T_a - lo < seg ? T_a - lo : seg;
    int m = (int)floor((double)retention * (double)len);
    total += m;
    if (variant == 0)
      for (int r = 0; r < m; ++r) { /* the r-th largest of the segment among those not taken yet */
        int best = -1;
        for (int t = lo; t < lo + len; ++t)
          if (!keep[t] && (best < 0 || key[t] > key[best])) best = t;
        keep[best] = 1;
      }
  }
  if (variant != 0)
    for (int r = 0; r < total; ++r) {
      int best = -1;
      for (int t = 0; t < T_a; ++t)
        if (!keep[t] && (best < 0 || key[t] > key[best])) best = t;
      keep[best] = 1;
    }
  int n = 0;
  for (int t = 0; t < T_a; ++t)
    if (keep[t]) kept[n++] = t;
  free(keep);
  return n;
}

/* Prefill placement with the fixed heads compressed token by token ("Prefill Compression"): anchor heads keep all
 * audio positions, the tidal table is filled as in wnwo_place_prefill_multi, and every fixed head h keeps the positions
 * wnwo_select_tokens picks from p_prefill[tau] = sum over the text queries and the head's q-heads of the attention
 * weight of tau (softmax over the whole prefix), with its own retention[h] (Eq. 1). */
int wnwo_place_prefill_tokens(Oracle *o, int seq, int layer, const uint16_t *k, const uint16_t *v, int n_tokens,
                              int audio_begin, int audio_end, const uint16_t *q_text, int n_q, const float *retention,
                              int seg, int variant) {
  if (!retention || seg < 1) return WNWO_ERR_ARG;
  int rc = place_multi(o, seq, layer, k, v, n_tokens, audio_begin, audio_end, q_text, n_q);
  if (rc) return rc;
  Seq *s = &o->seq[seq];
  const int T_a = s->T_a, T_t = s->T_t, Hkv = o->Hkv, d = o->d;
  if (s->C == 0) return WNWO_OK;
  unsigned char *all = (unsigned char *)malloc((size_t)s->C);
  double *out = (double *)malloc(sizeof(double) * d), *row = (double *)malloc(sizeof(double) * (size_t)(T_t + T_a));
  float *keyf = (float *)malloc(sizeof(float) * T_a);
  int *kept = (int *)malloc(sizeof(int) * T_a);
  memset(all, 1, (size_t)s->C);
  for (int h = 0; h < Hkv; ++h) {
    const int role = o->roles[layer * Hkv + h];
    if (role != ROLE_FIXED && !(role == ROLE_TIDAL && o->residency == 2)) continue;
    if (!(retention[h] >= 0.0f && retention[h] <= 1.0f)) { rc = WNWO_ERR_ARG; break; }
    const int idx = layer * Hkv + h;
    free(s->tok_mask[idx]); s->tok_mask[idx] = NULL; /* the scoring below sees every position */
    free(s->tok_score[idx]);
    double *p = s->tok_score[idx] = (double *)calloc((size_t)T_a, sizeof(double));
    for (int qi = 0; qi < n_q; ++qi)
      for (int j = 0; j < o->g; ++j) {
        attend(o, s, layer, h, q_text + ((size_t)qi * o->Hq + (size_t)(h * o->g + j)) * d, T_t, all, out, NULL, row);
        for (int t = 0; t < T_a; ++t) p[t] += row[T_t + t];
      }
    for (int t = 0; t < T_a; ++t) keyf[t] = (float)p[t];
    int n = wnwo_select_tokens(keyf, T_a, seg, retention[h], variant, kept);
    unsigned char *mask = (unsigned char *)calloc((size_t)T_a, 1);
    for (int i = 0; i < n; ++i) mask[kept[i]] = 1;
    s->tok_mask[idx] = mask;
  }
  free(all); free(out); free(row); free(keyf); free(kept);
  return rc;
}

int wnwo_get_token_scores(const Oracle *o, int seq, int layer, int kvh, double *out) {
  const Seq *s = &o->seq[seq];
  const double *p = s->tok_score ? s->tok_score[layer * o->Hkv + kvh] : NULL;
  if (!p) return WNWO_ERR_STATE;
  memcpy(out, p, sizeof(double) * s->T_a);
  return WNWO_OK;
}
/* kept positions of a fixed head placed token by token, ascending; returns their number (-1: chunk form) */
int wnwo_get_fixed_tokens(const Oracle *o, int seq, int layer, int kvh, int *pos) {
  const Seq *s = &o->seq[seq];
  const unsigned char *m = s->tok_mask ? s->tok_mask[layer * o->Hkv + kvh] : NULL;
  if (!m) return -1;
  int n = 0;
  for (int t = 0; t < s->T_a; ++t)
    if (m[t]) pos[n++] = t;
  return n;
}
int wnwo_set_fixed_tokens(Oracle *o, int seq, int layer, int kvh, const int *pos, int n) {
  Seq *s = &o->seq[seq];
  unsigned char *m = s->tok_mask ? s->tok_mask[layer * o->Hkv + kvh] : NULL;
  if (!m) return WNWO_ERR_STATE;
  memset(m, 0, (size_t)s->T_a);
  for (int i = 0; i < n; ++i) {
    if (pos[i] < 0 || pos[i] >= s->T_a) return WNWO_ERR_ARG;
    m[pos[i]] = 1;
  }
  return WNWO_OK;
}

int wnwo_place_prefill(Oracle *o, int seq, int layer, const uint16_t *k, const uint16_t *v, int n_tokens,
                       int audio_begin, int audio_end, const uint16_t *q_last) {
  return wnwo_place_prefill_multi(o, seq, layer, k, v, n_tokens, audio_begin, audio_end, q_last, 1);
}

/* ------------------------------------------------------------------ */
/* Streaming audio: the clip grows between decode steps                 */
/* ------------------------------------------------------------------ */
/* k, v: [L][n][Hkv][d] bf16 bits, the n new audio positions of every layer.  See the header for the reading. */
int wnwo_append_audio(Oracle *o, int seq, const uint16_t *k, const uint16_t *v, int n) {
  if (!o || seq < 0 || seq >= o->max_batch || n < 0 || (n > 0 && (!k || !v))) return WNWO_ERR_ARG;
  Seq *s = &o->seq[seq];
  if (o->in_step || s->placed_layers != o->L || o->residency != 0) return WNWO_ERR_STATE;
  if (s->T_a + n > o->max_audio) return WNWO_ERR_ARG;
  if (n == 0) return WNWO_OK;
  const int L = o->L, Hkv = o->Hkv, d = o->d;
  Seq old = *s, ns;
  memset(&ns, 0, sizeof(ns));
  int rc = alloc_seq(o, &ns, old.T_a + n, old.T_t);   /* the grown clip: C, and S by the slot rule */
  if (rc) { free_seq(o, &ns); return rc; }
  ns.placed_layers = L; ns.T_a_fixed = old.T_a_fixed; ns.steps = old.steps;
  ns.hits = old.hits; ns.misses = old.misses; ns.evictions = old.evictions;
  for (int l = 0; l < L; ++l) {
    memcpy(ns.txtK[l], old.txtK[l], (size_t)Hkv * old.T_cap * d * 2);
    memcpy(ns.txtV[l], old.txtV[l], (size_t)Hkv * old.T_cap * d * 2);
    for (int h = 0; h < Hkv; ++h) {
      uint16_t *dk = ns.audK[l] + (size_t)h * ns.T_a * d, *dv = ns.audV[l] + (size_t)h * ns.T_a * d;
      memcpy(dk, old.audK[l] + (size_t)h * old.T_a * d, (size_t)old.T_a * d * 2);
      memcpy(dv, old.audV[l] + (size_t)h * old.T_a * d, (size_t)old.T_a * d * 2);
      for (int i = 0; i < n; ++i) {
        const size_t src = (((size_t)l * n + i) * Hkv + h) * d;
        memcpy(dk + (size_t)(old.T_a + i) * d, k + src, (size_t)d * 2);
        memcpy(dv + (size_t)(old.T_a + i) * d, v + src, (size_t)d * 2);
      }
    }
    /* tables carry over; the slots the grown budget adds start empty (alloc_seq left them at -1, stamp 0) */
    for (int j = 0; j < old.S; ++j) {
      ns.slot_chunk[(size_t)l * ns.S + j] = old.slot_chunk[(size_t)l * old.S + j];
      ns.stamp[(size_t)l * ns.S + j] = old.stamp[(size_t)l * old.S + j];
    }
    for (int h = 0; h < Hkv; ++h) {   /* fixed sets are final */
      const int lh = l * Hkv + h;
      ns.fixed_n[lh] = old.fixed_n[lh];
      for (int j = 0; j < old.fixed_n[lh]; ++j) ns.fixed_set[(size_t)lh * ns.S + j] = old.fixed_set[(size_t)lh * old.S + j];
      for (int c = 0; c < old.C; ++c) ns.pre[(size_t)lh * ns.C + c] = old.pre[(size_t)lh * old.C + c];
      if (old.tok_mask && old.tok_mask[lh]) {   /* a head placed token by token keeps its positions; later ones are not kept */
        ns.tok_mask[lh] = (unsigned char *)calloc((size_t)ns.T_a, 1);
        if (!ns.tok_mask[lh]) { free_seq(o, &ns); return WNWO_ERR_OOM; }
        memcpy(ns.tok_mask[lh], old.tok_mask[lh], (size_t)old.T_a);
      }
    }
    for (int c = 0; c < old.C; ++c) ns.score_sum[(size_t)l * ns.C + c] = old.score_sum[(size_t)l * old.C + c];
    for (int r = 0; r < o->topk; ++r) ns.sel[(size_t)l * o->topk + r] = old.sel[(size_t)l * o->topk + r];
    ns.n_sel[l] = old.n_sel[l];
  }
  free_seq(o, &old);
  *s = ns;
  return WNWO_OK;
}

/* ------------------------------------------------------------------ */
/* Decode step                                                          */
/* ------------------------------------------------------------------ */

int wnwo_step_begin(Oracle *o, const int *active, int n_active) {
  if (!o || !active || n_active < 1 || n_active > o->max_batch) return WNWO_ERR_ARG;
  if (o->in_step) return WNWO_ERR_STATE;
  for (int i = 0; i < n_active; ++i) {
    int b = active[i];
    if (b < 0 || b >= o->max_batch) return WNWO_ERR_ARG;
    if (o->seq[b].placed_layers != o->L) return WNWO_ERR_STATE;
    for (int j = 0; j < i; ++j) if (active[j] == b) return WNWO_ERR_ARG;
  }
  memcpy(o->active, active, sizeof(int) * n_active);
  o->n_active = n_active; o->in_step = 1; o->next_layer = 0; o->appended = -1;
  if (o->sharded) /* a layer whose anchor heads all sit in other shards contributes a zero partial sum */
    for (int i = 0; i < n_active; ++i) {
      Seq *s = &o->seq[active[i]];
      memset(s->score_sum, 0, sizeof(double) * (size_t)o->L * (size_t)(s->C > 0 ? s->C : 1));
    }
  return WNWO_OK;
}

/* q: [n_active][Hq][d]; k_new,v_new: [n_active][Hkv][d] or NULL; out: [n_active][Hq][d] double. */
int wnwo_decode_layer(Oracle *o, int layer, const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new, double *out) {
  if (!o || !q || !out || (k_new == NULL) != (v_new == NULL)) return WNWO_ERR_ARG;
  if (!o->in_step || layer != o->next_layer) return WNWO_ERR_STATE;
  const int has_new = k_new != NULL;
  if (o->appended >= 0 && o->appended != has_new) return WNWO_ERR_STATE;
  const int Hq = o->Hq, Hkv = o->Hkv, d = o->d, g = o->g;
  for (int i = 0; i < o->n_active; ++i)
    if (has_new && o->seq[o->active[i]].T_t + 1 > o->seq[o->active[i]].T_cap) return WNWO_ERR_ARG;
  o->appended = has_new;
  const int anchor_layer = layer_has(o, layer, ROLE_ANCHOR);
  for (int i = 0; i < o->n_active; ++i) {
    Seq *s = &o->seq[o->active[i]];
    int T_t = s->T_t;
    if (has_new) { /* generated tokens are kept in full: append to the text region */
      for (int h = 0; h < Hkv; ++h) {
        size_t off = ((size_t)h * s->T_cap + (size_t)T_t) * d;
        memcpy(s->txtK[layer] + off, k_new + ((size_t)i * Hkv + h) * d, (size_t)d * 2);
        memcpy(s->txtV[layer] + off, v_new + ((size_t)i * Hkv + h) * d, (size_t)d * 2);
      }
      T_t += 1;
    }
    const int C = s->C;
    double *mass = (double *)calloc((size_t)Hq * (size_t)(C > 0 ? C : 1), sizeof(double));
#pragma omp parallel for schedule(dynamic, 1)
    for (int hq = 0; hq < Hq; ++hq) {
      int kvh = hq / g;
      unsigned char *allowed = (unsigned char *)malloc((size_t)(C > 0 ? C : 1));
      allowed_for(o, s, layer, kvh, allowed);
      int is_anchor = o->roles[layer * Hkv + kvh] == ROLE_ANCHOR;
      attend(o, s, layer, kvh, q + ((size_t)i * Hq + hq) * d, T_t, allowed, out + ((size_t)i * Hq + hq) * d,
             is_anchor ? mass + (size_t)hq * C : NULL, NULL);
      free(allowed);
    }
    if (anchor_layer) { /* Eq. 2 summed over tau in c, over this layer's anchor q-heads, in head order */
      double *sc = s->score_sum + (size_t)layer * C;
      for (int c = 0; c < C; ++c) sc[c] = 0.0;
      for (int hq = 0; hq < Hq; ++hq)
        if (o->roles[layer * Hkv + hq / g] == ROLE_ANCHOR)
          for (int c = 0; c < C; ++c) sc[c] += mass[(size_t)hq * C + c];
    }
    free(mass);
  }
  o->next_layer = layer + 1;
  return WNWO_OK;
}

/* Selection + table update of every tidal layer, from this step's scores. */
int wnwo_step_end(Oracle *o) {
  if (!o || !o->in_step || o->next_layer != o->L) return WNWO_ERR_STATE;
  for (int i = 0; i < o->n_active; ++i) {
    Seq *s = &o->seq[o->active[i]];
    const int C = s->C, S = s->S;
    if (C > 0) {
      int *lens = (int *)malloc(sizeof(int) * C);
      float *sf = (float *)malloc(sizeof(float) * C);
      int *pc = (int *)malloc(sizeof(int) * o->topk), *ps = (int *)malloc(sizeof(int) * o->topk),
          *ev = (int *)malloc(sizeof(int) * o->topk);
      for (int c = 0; c < C; ++c) lens[c] = chunk_len(o, s, c);
      double *glob = (double *)calloc((size_t)C, sizeof(double));
      if (o->scope == 1) /* Eq. 2: one accumulator over all anchor (layer, q-head) pairs of the step */
        for (int a = 0; a < o->L; ++a)
          if (o->anchor_layer[a])
            for (int c = 0; c < C; ++c) glob[c] += s->score_sum[(size_t)a * C + c];
      int *segs = (int *)malloc(sizeof(int) * 2 * o->topk), *rel = (int *)malloc(sizeof(int) * (size_t)(S > 0 ? S : 1));
      int *pg = (int *)malloc(sizeof(int) * 2 * o->topk), *pj = (int *)malloc(sizeof(int) * 2 * o->topk);
      for (int l = 0; l < o->L; ++l) {
        s->n_sel[l] = 0;
        if (o->src[l] < 0) continue;
        const double *sc = o->scope == 1 ? glob : s->score_sum + (size_t)o->src[l] * C;
        for (int c = 0; c < C; ++c) sf[c] = (float)sc[c];
        if (o->residency >= 1) { /* overlapping chunks, permanent base, lag-delta release */
          int n_sel = 0, n_rel = 0, hits = 0;
          int n_seg = wnwo_select_segments(sf, lens, C, o->topk, s->sel + (size_t)l * o->topk, &n_sel, segs);
          s->n_sel[l] = n_sel;
          int n = wnwo_lag_update(s->slot_chunk + (size_t)l * S, s->stamp + (size_t)l * S, s->S_base, S, segs, n_seg, s->steps,
                                  o->delta, pg, pj, rel, &n_rel, &hits);
          s->hits += hits; s->misses += n; s->evictions += n_rel;
          continue;
        }
        int k = o->topk < S ? o->topk : S;
        k = wnwo_topk(sf, lens, C, k, s->sel + (size_t)l * o->topk);
        s->n_sel[l] = k;
        int hits = 0;
        int n = wnwo_table_update(s->slot_chunk + (size_t)l * S, s->stamp + (size_t)l * S, S, s->sel + (size_t)l * o->topk, k,
                                  s->steps, o->topk, pc, ps, ev, &hits);
        s->hits += hits; s->misses += n;
        for (int j = 0; j < n; ++j) s->evictions += ev[j] >= 0;
      }
      free(lens); free(sf); free(pc); free(ps); free(ev); free(glob); free(segs); free(rel); free(pg); free(pj);
    }
    s->steps += 1;
    if (o->appended == 1) s->T_t += 1;
  }
  o->in_step = 0;
  return WNWO_OK;
}

/* ------------------------------------------------------------------ */
/* Inspection and lock-step helpers                                     */
/* ------------------------------------------------------------------ */

/* Head-sharded serving: the chunk scores of `layer` summed over all shards replace this shard's partial sum, between
 * the last layer of a step and wnwo_step_end. */
int wnwo_set_chunk_scores(Oracle *o, int seq, int layer, const double *scores) {
  if (!o || !scores || seq < 0 || seq >= o->max_batch || layer < 0 || layer >= o->L) return WNWO_ERR_ARG;
  if (!o->in_step || o->next_layer != o->L) return WNWO_ERR_STATE;
  Seq *s = &o->seq[seq];
  for (int c = 0; c < s->C; ++c) s->score_sum[(size_t)layer * s->C + c] = scores[c];
  return WNWO_OK;
}

int wnwo_get_dims(const Oracle *o, int seq, int *T_a, int *T_t, int *C, int *S) {
  if (!o || seq < 0 || seq >= o->max_batch || o->seq[seq].placed_layers == 0) return WNWO_ERR_STATE;
  const Seq *s = &o->seq[seq];
  *T_a = s->T_a; *T_t = s->T_t; *C = s->C; *S = s->S;
  return WNWO_OK;
}
int wnwo_get_base_slots(const Oracle *o, int seq, int *S_base) {
  if (!o || seq < 0 || seq >= o->max_batch || o->seq[seq].placed_layers == 0) return WNWO_ERR_STATE;
  *S_base = o->seq[seq].S_base;
  return WNWO_OK;
}
int wnwo_get_chunk_scores(const Oracle *o, int seq, int layer, double *scores) {
  const Seq *s = &o->seq[seq];
  memcpy(scores, s->score_sum + (size_t)layer * s->C, sizeof(double) * s->C);
  return WNWO_OK;
}
int wnwo_get_prefill_scores(const Oracle *o, int seq, int layer, int kvh, double *scores) {
  const Seq *s = &o->seq[seq];
  memcpy(scores, s->pre + ((size_t)layer * o->Hkv + kvh) * s->C, sizeof(double) * s->C);
  return WNWO_OK;
}
int wnwo_get_selected(const Oracle *o, int seq, int layer, int *sel) {
  const Seq *s = &o->seq[seq];
  memcpy(sel, s->sel + (size_t)layer * o->topk, sizeof(int) * o->topk);
  return s->n_sel[layer];
}
int wnwo_get_residency(const Oracle *o, int seq, int layer, int *slot_chunk, long long *stamp) {
  const Seq *s = &o->seq[seq];
  memcpy(slot_chunk, s->slot_chunk + (size_t)layer * s->S, sizeof(int) * s->S);
  if (stamp) memcpy(stamp, s->stamp + (size_t)layer * s->S, sizeof(long long) * s->S);
  return WNWO_OK;
}
int wnwo_set_residency(Oracle *o, int seq, int layer, const int *slot_chunk, const long long *stamp) {
  Seq *s = &o->seq[seq];
  memcpy(s->slot_chunk + (size_t)layer * s->S, slot_chunk, sizeof(int) * s->S);
  memcpy(s->stamp + (size_t)layer * s->S, stamp, sizeof(long long) * s->S);
  return WNWO_OK;
}
int wnwo_get_fixed_set(const Oracle *o, int seq, int layer, int kvh, int *chunks) {
  const Seq *s = &o->seq[seq];
  int n = s->fixed_n[layer * o->Hkv + kvh];
  memcpy(chunks, s->fixed_set + ((size_t)layer * o->Hkv + kvh) * s->S, sizeof(int) * n);
  return n;
}
int wnwo_set_fixed_set(Oracle *o, int seq, int layer, int kvh, const int *chunks, int n) {
  Seq *s = &o->seq[seq];
  if (n > s->S) return WNWO_ERR_ARG;
  memcpy(s->fixed_set + ((size_t)layer * o->Hkv + kvh) * s->S, chunks, sizeof(int) * n);
  s->fixed_n[layer * o->Hkv + kvh] = n;
  return WNWO_OK;
}
int wnwo_get_stats(const Oracle *o, int seq, long long *hits, long long *misses, long long *evictions) {
  const Seq *s = &o->seq[seq];
  *hits = s->hits; *misses = s->misses; *evictions = s->evictions;
  return WNWO_OK;
}

/* The probability row of one query head over [text | audio] as the oracle sees
 * it now (no state change, no append).  p_row: [T_t + T_a]; out: [d]. */
int wnwo_attention_row(const Oracle *o, int seq, int layer, int q_head, const uint16_t *q, double *p_row, double *out) {
  if (!o || seq < 0 || seq >= o->max_batch || layer < 0 || layer >= o->L || q_head < 0 || q_head >= o->Hq) return WNWO_ERR_ARG;
  const Seq *s = &o->seq[seq];
  if (s->placed_layers <= layer) return WNWO_ERR_STATE;
  unsigned char *allowed = (unsigned char *)malloc((size_t)(s->C > 0 ? s->C : 1));
  allowed_for(o, s, layer, q_head / o->g, allowed);
  attend(o, s, layer, q_head / o->g, q, s->T_t, allowed, out, NULL, p_row);
  free(allowed);
  return WNWO_OK;
}
