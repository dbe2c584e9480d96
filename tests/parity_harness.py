"""Lock-step parity driver: the CUDA path (through the C ABI binding) against the CPU oracle on the same seeded bits.

Staged parity, because selected indices must match bit-exactly while the scores they derive from are floating point:
  (i)   scores (decode chunk scores, prefill scores): |gpu - oracle| <= 1e-4 * |oracle| + 1e-8;
  (ii)  the oracle's top-k and table update, run on the GPU's own fp32 scores and the GPU's previous table, must
        reproduce the GPU's selection, table and stamps bit-exactly;
  (iii) the oracle, selecting from its own fp64 scores, must agree as well; a disagreement is accepted only if the
        ranking keys at the selection boundary are within 2e-4 relative (a near-tie), is counted, and the oracle then
        adopts the GPU's table so the trajectories stay aligned.
Attention outputs: max |gpu - oracle| <= 2e-2 (bf16 outputs of O(1) magnitude).
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2608_22704_b200 as wnw
from helpers import bf16_bits_to_f64, dequantised_tidal_bits, make_oracle
from oracle import wnw_oracle as wo
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, Workload
from workloads.synth import bf16_bits

OUT_TOL = 2e-2
SCORE_RTOL, SCORE_ATOL = 1e-4, 1e-8
TIE_RTOL = 2e-4


def chunk_lens(T_a, chunk):
    C = -(-T_a // chunk)
    return np.array([min(chunk, T_a - c * chunk) for c in range(C)], np.int32)


def assert_scores_close(gpu, ref, what):
    gpu = np.asarray(gpu, np.float64); ref = np.asarray(ref, np.float64)
    err = np.abs(gpu - ref)
    bound = SCORE_RTOL * np.abs(ref) + SCORE_ATOL
    assert (err <= bound).all(), f"{what}: worst rel err {(err / np.maximum(np.abs(ref), 1e-30)).max():.3e}"


def near_tie(scores64, lens, sel_a, sel_b):
    """True if the two selections differ only across a near-tie of the ranking key."""
    key = (np.asarray(scores64, np.float64) / lens)
    diff = set(sel_a) ^ set(sel_b)
    if not diff:   # same set, different order: the swapped ranks must be near-ties
        diff = {a for a, b in zip(sel_a, sel_b) if a != b} | {b for a, b in zip(sel_a, sel_b) if a != b}
    ks = key[sorted(diff)]
    return (ks.max() - ks.min()) <= TIE_RTOL * max(ks.max(), 1e-30)


class Lockstep:
    def __init__(self, w: Workload, seed=0, device="cuda:0", recall_mode=0, gen_device=None, oracle_seqs=None,
                 score_scope=0, residency=0, evict_lag=3, token_retention=None, token_seg=25, token_variant=0, kv_fp8=False):
        self.w = w
        # e4m3 storage of the tidal tier: the library gets the plain bf16 prefix and the format flag; the oracle, which knows
        # nothing of storage formats, gets the values the stored bytes decode to (helpers.dequantised_tidal_bits)
        self.kv_fp8 = kv_fp8
        # token-granular compression of fixed heads: retention [n_layers][n_kv_heads], segment size, variant
        self.tok_ret = None if token_retention is None else np.asarray(token_retention, np.float32)
        self.tok_seg, self.tok_variant = token_seg, token_variant
        self.dev = torch.device(device)
        self.syn = Synth(w, seed=seed, device=gen_device or "cpu")
        self.oracle_seqs = list(range(w.batch)) if oracle_seqs is None else list(oracle_seqs)
        self.scope = score_scope
        self.residency, self.evict_lag = residency, evict_lag
        self.o = make_oracle(w, score_scope=score_scope, residency=residency, evict_lag=evict_lag)
        self.h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(max(w.audio_lens), 0),
                                w.text_capacity, w.chunk, w.budget, w.roles, topk=w.topk, device=self.dev.index or 0,
                                recall_mode=recall_mode, score_scope=score_scope, residency=residency, evict_lag=evict_lag,
                                tidal_kv_format=wnw.WNW_TIDAL_KV_FP8_E4M3 if kv_fp8 else wnw.WNW_TIDAL_KV_BF16)
        self.kept = {}
        self.tok_kept = {}
        self.near_ties = 0
        self.max_out_err = 0.0
        self.dec = {}
        self.step = 0
        self._steps = {}
        self.expected_recall_bytes = 0

    def close(self):
        if self.h:
            wnw.wnw_destroy(self.h); self.h = None
        self.o.close()

    # ------------------------------------------------------------------ prefill
    def prefill(self, check_slots=True):
        w = self.w
        for b in range(w.batch):
            for l in range(w.n_layers):
                p = self.syn.prefill(b, l)
                qname = "q_text" if "q_text" in p else "q_last"     # all text queries when the workload has several
                k, v, ql = (p[n].to(self.dev) for n in ("k", "v", qname))
                if self.tok_ret is not None:
                    if ql.dim() == 2:
                        ql = ql[None]
                    wnw.wnw_place_prefill_tokens(self.h, b, l, k, v, p["audio_begin"], p["audio_end"], ql, self.tok_ret[l],
                                                 self.tok_seg, self.tok_variant)
                else:
                    wnw.wnw_place_prefill(self.h, b, l, k, v, p["audio_begin"], p["audio_end"], ql)
                if self.syn.device.type == "cuda":
                    torch.cuda.synchronize(self.dev)   # the generator's buffers are released right after
                if b in self.oracle_seqs:
                    kb, vb = bf16_bits(p["k"]), bf16_bits(p["v"])
                    if self.kv_fp8:
                        kb, vb = dequantised_tidal_bits(kb, vb, w.roles[l], p["audio_begin"], p["audio_end"], w.chunk)
                    if self.tok_ret is not None:
                        self.o.place_prefill_tokens(b, l, kb, vb, p["audio_begin"], p["audio_end"], bf16_bits(p[qname]),
                                                    self.tok_ret[l], self.tok_seg, self.tok_variant)
                        self.check_token_sets(b, l, p["audio_end"] - p["audio_begin"])
                    else:
                        self.o.place_prefill(b, l, kb, vb, p["audio_begin"], p["audio_end"], bf16_bits(p[qname]))
                    self.kept[(b, l)] = (kb[p["audio_begin"]:p["audio_end"]], vb[p["audio_begin"]:p["audio_end"]])
        wnw.wnw_sync(self.h)
        for b in self.oracle_seqs:
            T_a, T_t, C, S = wnw.wnw_get_seq_dims(self.h, b)
            assert (T_a, T_t, C, S) == self.o.dims(b)
            if C == 0:
                continue
            lens = chunk_lens(T_a, w.chunk)
            S_all, S = S, wnw.wnw_get_base_slots(self.h, b)      # the prefill placement fills the permanent slots
            assert S == self.o.base_slots(b)
            for l in range(w.n_layers):
                tid_sum = np.zeros(C, np.float32)
                any_tid = False
                for h in range(w.n_kv_heads):
                    role = w.roles[l, h]
                    if role == ROLE_ANCHOR:
                        continue
                    g_pre = wnw.wnw_get_prefill_scores(self.h, b, l, h)
                    assert_scores_close(g_pre, self.o.prefill_scores(b, l, h), f"prefill scores b{b} l{l} h{h}")
                    if role == ROLE_FIXED and self.tok_ret is not None:
                        continue                                   # kept positions, checked right after the placement
                    if role == ROLE_FIXED:
                        g_set = wnw.wnw_get_fixed_set(self.h, b, l, h)
                        assert g_set.tolist() == wo.topk(g_pre, lens, S).tolist(), f"fixed set (ii) b{b} l{l} h{h}"
                        o_set = self.o.fixed_set(b, l, h)
                        if g_set.tolist() != o_set.tolist():
                            assert near_tie(self.o.prefill_scores(b, l, h), lens, g_set.tolist(), o_set.tolist())
                            self.near_ties += 1
                            self.o.set_fixed_set(b, l, h, g_set)
                    else:
                        tid_sum = (tid_sum + g_pre).astype(np.float32); any_tid = True
                if any_tid:
                    g_tab, g_stamp = wnw.wnw_get_residency(self.h, b, l)
                    want = wo.topk(tid_sum, lens, S)
                    assert g_tab.tolist() == want.tolist() + [-1] * (S_all - S), f"tidal table (ii) b{b} l{l}"
                    assert g_stamp.tolist() == [-1 - r for r in range(S)] + [0] * (S_all - S)
                    o_tab, o_stamp = self.o.residency(b, l)
                    if g_tab.tolist() != o_tab.tolist():
                        o_sum = sum(self.o.prefill_scores(b, l, h) for h in range(w.n_kv_heads) if w.roles[l, h] == ROLE_TIDAL)
                        assert near_tie(o_sum, lens, g_tab[:S].tolist(), o_tab[:S].tolist())
                        self.near_ties += 1
                        self.o.set_residency(b, l, g_tab, g_stamp)
                    if check_slots:
                        self.check_slot_bytes(b, l)

    def check_token_sets(self, b, l, T_a):
        """Token-compressed fixed heads of (b, l), right after their placement: (i) per-position scores close,
        (ii) the oracle's selection on the GPU's fp32 scores reproduces the GPU's kept positions bit-exactly,
        (iii) the oracle's own set agrees or differs only across near-ties (then it adopts the GPU's)."""
        w = self.w
        if T_a == 0:
            return
        for h in range(w.n_kv_heads):
            if w.roles[l, h] != ROLE_FIXED and not (w.roles[l, h] == ROLE_TIDAL and self.residency == 2):
                continue
            g_p = wnw.wnw_get_token_scores(self.h, b, l, h)
            o_p = self.o.token_scores(b, l, h)
            assert_scores_close(g_p, o_p, f"token scores b{b} l{l} h{h}")
            g_pos = wnw.wnw_get_fixed_tokens(self.h, b, l, h)
            want = wo.select_tokens(g_p, self.tok_seg, float(self.tok_ret[l, h]), self.tok_variant)
            assert g_pos.tolist() == want.tolist(), f"kept positions (ii) b{b} l{l} h{h}"
            o_pos = self.o.fixed_tokens(b, l, h)
            if g_pos.tolist() != o_pos.tolist():
                assert len(g_pos) == len(o_pos)
                diff = sorted(set(g_pos.tolist()) ^ set(o_pos.tolist()))
                groups = {}
                for t in diff:
                    groups.setdefault(t // self.tok_seg if self.tok_variant == 0 else 0, []).append(t)
                for ts in groups.values():
                    ks = o_p[ts]
                    assert ks.max() - ks.min() <= TIE_RTOL * max(ks.max(), 1e-30), f"kept positions b{b} l{l} h{h}: {ts}"
                self.near_ties += 1
                self.o.set_fixed_tokens(b, l, h, g_pos)
            self.tok_kept[(b, l, h)] = g_pos

    def check_slot_bytes(self, b, l):
        """Slot contents are an exact copy of the source K,V of the chunk the table says is there."""
        w = self.w
        tab, _ = wnw.wnw_get_residency(self.h, b, l)
        T_a = w.audio_lens[b]
        kb, vb = self.kept[(b, l)]
        for h in range(w.n_kv_heads):
            if w.roles[l, h] != ROLE_TIDAL:
                continue
            for j, c in enumerate(tab.tolist()):
                if c < 0:
                    continue
                n = min(w.chunk, T_a - c * w.chunk)
                order = np.arange(n)
                if self.residency == 2:       # token-granular base: the positions outside the base first, the kept ones after
                    kept = set(self.tok_kept[(b, l, h)].tolist())
                    inb = np.array([c * w.chunk + r in kept for r in range(n)])
                    order = np.concatenate([np.nonzero(~inb)[0], np.nonzero(inb)[0]])
                for which, src in ((0, kb), (1, vb)):
                    rows = wnw.wnw_get_slot_kv(self.h, b, l, h, j, which, w.chunk, w.head_dim)
                    assert np.array_equal(rows[:n], src[c * w.chunk:c * w.chunk + n, h][order]), f"slot bytes b{b} l{l} h{h} slot{j}"

    # ------------------------------------------------------------------ decode
    def _dec(self, b, l):
        if (b, l) not in self.dec:
            self.dec[(b, l)] = self.syn.decode(b, l)
        return self.dec[(b, l)]

    def decode_step(self, t=None, append=True, active=None, check_slots=False, graph=False):
        """One lock-step decode step.  graph=True replays a captured CUDA graph of the step (captured on first use)
        from static input buffers instead of issuing the layers eagerly."""
        w = self.w
        t = self.step if t is None else t
        active = list(range(w.batch)) if active is None else list(active)
        o_active = [b for b in active if b in self.oracle_seqs]
        prev_tab = {(b, l): wnw.wnw_get_residency(self.h, b, l) for b in o_active for l in range(w.n_layers)
                    if (w.roles[l] == ROLE_TIDAL).any()}
        steps_before = {b: self._steps.get(b, 0) for b in active}
        if o_active:
            self.o.step_begin(o_active)
        outs = []
        qs = [torch.stack([self._dec(b, l)["q"][t] for b in active]).to(self.dev) for l in range(w.n_layers)]
        kns = [torch.stack([self._dec(b, l)["k_new"][t] for b in active]).to(self.dev) if append else None for l in range(w.n_layers)]
        vns = [torch.stack([self._dec(b, l)["v_new"][t] for b in active]).to(self.dev) if append else None for l in range(w.n_layers)]
        if graph:
            if getattr(self, "_graph", None) is None:
                self._gstream = torch.cuda.Stream(device=self.dev)
                self._gq = [torch.empty_like(x) for x in qs]
                self._gkn = [torch.empty_like(x) if x is not None else None for x in kns]
                self._gvn = [torch.empty_like(x) if x is not None else None for x in vns]
                self._gout = [torch.empty_like(x) for x in qs]
                torch.cuda.synchronize(self.dev)
                wnw.wnw_graph_begin(self.h, active, self._gstream)
                wnw.wnw_step_begin(self.h, active)
                for l in range(w.n_layers):
                    wnw.wnw_decode_layer(self.h, l, self._gq[l], self._gkn[l], self._gvn[l], self._gout[l], stream=self._gstream)
                wnw.wnw_step_end(self.h, stream=self._gstream)
                wnw.wnw_graph_end(self.h, self._gstream)
                self._graph = True
            # the inputs were produced on the current stream: the replay stream must not read them earlier
            self._gstream.wait_stream(torch.cuda.current_stream(self.dev))
            with torch.cuda.stream(self._gstream):
                for l in range(w.n_layers):
                    self._gq[l].copy_(qs[l])
                    if append:
                        self._gkn[l].copy_(kns[l]); self._gvn[l].copy_(vns[l])
            wnw.wnw_graph_launch(self.h, self._gstream)
            self._gstream.synchronize()
        else:
            wnw.wnw_step_begin(self.h, active)
        for l in range(w.n_layers):
            q, kn, vn = qs[l], kns[l], vns[l]
            if graph:
                out = self._gout[l]
            else:
                out = torch.empty_like(q)
                wnw.wnw_decode_layer(self.h, l, q, kn, vn, out)
            outs.append((q, kn, vn, out))
            if o_active:
                idx = [active.index(b) for b in o_active]
                qb = bf16_bits(q.cpu())[idx]
                knb = bf16_bits(kn.cpu())[idx] if append else None
                vnb = bf16_bits(vn.cpu())[idx] if append else None
                ref = self.o.decode_layer(l, qb, knb, vnb)
                got = bf16_bits_to_f64(bf16_bits(out.cpu()))[idx]
                err = np.abs(got - ref).max()
                self.max_out_err = max(self.max_out_err, float(err))
                if not err <= OUT_TOL:
                    bad = np.argwhere(~(np.abs(got - ref) <= OUT_TOL))
                    heads = sorted({(int(x[0]), int(x[1]) // (w.n_q_heads // w.n_kv_heads)) for x in bad})
                    raise AssertionError(f"attention output step {t} layer {l}: max abs err {err:.4f}; (seq, kv head, role) "
                                         f"{[(i, h, int(w.roles[l, h])) for i, h in heads][:8]}")
        if not graph:
            wnw.wnw_step_end(self.h)
        wnw.wnw_sync(self.h)
        if o_active:
            self.o.step_end()
        for b in o_active:
            T_a, _, C, S = self.o.dims(b)
            if C == 0:
                continue
            lens = chunk_lens(T_a, w.chunk)
            g_scores = {}
            for l in range(w.n_layers):
                if (w.roles[l] == ROLE_ANCHOR).any():
                    g_scores[l] = wnw.wnw_get_chunk_scores(self.h, b, l)
                    assert_scores_close(g_scores[l], self.o.chunk_scores(b, l), f"chunk scores step {t} b{b} l{l}")
            for l in range(w.n_layers):
                if not (w.roles[l] == ROLE_TIDAL).any():
                    continue
                if self.scope == 1:   # Eq. 2 as printed: fp32 sum over the anchor layers, in layer order
                    rank_g = np.zeros(C, np.float32)
                    rank_o = np.zeros(C, np.float64)
                    for a in sorted(g_scores):
                        rank_g = (rank_g + g_scores[a].astype(np.float32)).astype(np.float32)
                        rank_o += self.o.chunk_scores(b, a)
                else:
                    src = self.o.score_source(l)
                    rank_g, rank_o = g_scores[src], self.o.chunk_scores(b, src)
                k = min(w.topk, S)
                g_sel = wnw.wnw_get_selected(self.h, b, l)
                g_tab, g_stamp = wnw.wnw_get_residency(self.h, b, l)
                # (ii) oracle logic on GPU scores and the GPU's previous table
                tab, stamp = prev_tab[(b, l)][0].copy(), prev_tab[(b, l)][1].copy()
                if self.residency >= 1:   # overlapping chunks, permanent base, lag-delta release
                    want_sel, segs = wo.select_segments(rank_g, lens, w.topk)
                    assert g_sel.tolist() == want_sel.tolist(), f"selection (ii) step {t} b{b} l{l}"
                    plan, _, _ = wo.lag_update(tab, stamp, wnw.wnw_get_base_slots(self.h, b), segs, steps_before[b], self.evict_lag)
                    if C > 1:                  # the ranking the near-tie check looks at: chunk sums and lengths
                        rank_o, lens_tie = rank_o[:-1] + rank_o[1:], lens[:-1] + lens[1:]
                else:
                    want_sel = wo.topk(rank_g, lens, k)
                    assert g_sel.tolist() == want_sel.tolist(), f"selection (ii) step {t} b{b} l{l}"
                    plan, _ = wo.table_update(tab, stamp, want_sel, steps_before[b], w.topk)
                n_tid = int((w.roles[l] == ROLE_TIDAL).sum())
                self.expected_recall_bytes += len(plan) * n_tid * 2 * (-(-w.chunk // 16) * 16) * w.head_dim * (1 if self.kv_fp8 else 2)   # blocks are stored padded to 16 rows
                assert g_tab.tolist() == tab.tolist(), f"table (ii) step {t} b{b} l{l}"
                assert g_stamp.tolist() == stamp.tolist(), f"stamps (ii) step {t} b{b} l{l}"
                # (iii) oracle on its own scores
                o_sel = self.o.selected(b, l)
                o_tab, o_stamp = self.o.residency(b, l)
                if o_sel.tolist() != g_sel.tolist() or o_tab.tolist() != g_tab.tolist() or o_stamp.tolist() != g_stamp.tolist():
                    assert near_tie(rank_o, lens_tie if self.residency >= 1 and C > 1 else lens, g_sel.tolist(), o_sel.tolist()), \
                        f"selection differs beyond a near-tie, step {t} b{b} l{l}: gpu {g_sel} oracle {o_sel}"
                    self.near_ties += 1
                    self.o.set_residency(b, l, g_tab, g_stamp)
                if check_slots:
                    self.check_slot_bytes(b, l)
        for b in active:
            self._steps[b] = steps_before[b] + 1
        self.step = t + 1
        return outs

    def check_stats(self):
        """Hit/miss/eviction counters agree with the oracle's when the oracle follows every sequence."""
        if sorted(self.oracle_seqs) != list(range(self.w.batch)) or self.near_ties:
            return
        g = wnw.wnw_get_stats(self.h)
        o = {"hits": 0, "misses": 0, "evictions": 0}
        for b in range(self.w.batch):
            s = self.o.stats(b)
            for k in o:
                o[k] += s[k]
        assert (g["hits"], g["misses"], g["evictions"]) == (o["hits"], o["misses"], o["evictions"])
        assert g["recall_bytes"] == self.expected_recall_bytes
