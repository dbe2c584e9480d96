"""Pins of the oracle's token-granular prefill compression of fixed heads (CPU only).

What is pinned: Eq. 1 (retention schedule) against its closed form; the per-segment top-floor(retention * n_s) rule
of "Prefill Compression" and the global top-k variant of the ablation against numpy sorts, hand-worked examples and
the invariants the paper states (every segment keeps its quota, so none is wholly evicted; both variants keep the
same number of positions); the per-position prefill score against a separate numpy softmax; and the decode output of
a compressed fixed head against numpy attention over exactly [text | kept positions].
"""
import math

import numpy as np
import pytest

from helpers import bf16_bits_to_f64, dense_attention, make_oracle
from oracle import wnw_oracle as wo
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, tiny_custom
from workloads.synth import bf16_bits

A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


# ---------------------------------------------------------------- Eq. 1
def test_retention_schedule_closed_form():
    s = np.array([0.0, 0.1, 0.25, 0.5, 1.0])
    assert wo.retention_schedule(s, 2.0).tolist() == [0.0, 0.2, 0.5, 1.0, 1.0]      # clipped at 1
    assert wo.retention_schedule(s, 0.0).tolist() == [0.0] * 5
    assert wo.retention_schedule(s, 1.0).tolist() == s.tolist()
    # large lambda: every head saturates, nothing is left to recall
    assert wo.retention_schedule(s[1:], 1e6).tolist() == [1.0] * 4
    # below saturation the schedule is proportional to the importance
    r = wo.retention_schedule(s, 0.7)
    assert r == pytest.approx(0.7 * s, abs=1e-15)


# ---------------------------------------------------------------- per-segment top-k and the global variant
def test_select_tokens_hand_example():
    """Segments of 3: [0.1 0.5 0.2 | 0.9 0.3 0.3 | 0.05], retention 0.67 -> floor(2.01) = 2 per full segment, floor(0.67) = 0
    in the tail.  Segment 0 keeps positions 1, 2; segment 1 keeps 3 and the EARLIER of the two equal keys (4)."""
    key = [0.1, 0.5, 0.2, 0.9, 0.3, 0.3, 0.05]
    assert wo.select_tokens(key, 3, 0.67, 0).tolist() == [1, 2, 3, 4]
    # global variant: same total (4), best of the whole head: 0.9, 0.5, 0.3, 0.3
    assert wo.select_tokens(key, 3, 0.67, 1).tolist() == [1, 3, 4, 5]
    assert wo.select_tokens(key, 3, 1.0, 0).tolist() == list(range(7))
    assert wo.select_tokens(key, 3, 0.0, 0).tolist() == []
    assert wo.select_tokens(key, 3, 0.33, 0).tolist() == []            # floor(0.99) = 0 everywhere
    assert wo.select_tokens(key, 3, 0.34, 0).tolist() == [1, 3]        # one per full segment, none in the tail
    assert wo.select_tokens([], 3, 0.5, 0).tolist() == []


@pytest.mark.parametrize("T_a,seg,ret", [(150, 25, 0.2), (1000, 50, 0.37), (77, 25, 0.5), (64, 64, 0.1), (30, 7, 0.9)])
def test_select_tokens_matches_numpy_sort(T_a, seg, ret):
    rng = np.random.RandomState(T_a + seg)
    key = rng.rand(T_a).astype(np.float32)
    key[rng.randint(0, T_a, T_a // 5)] = key[0]          # plenty of exact ties
    r32 = float(np.float32(ret))
    want, total = [], 0
    for lo in range(0, T_a, seg):
        k = key[lo:lo + seg]
        m = int(math.floor(r32 * len(k)))
        total += m
        order = np.argsort(-k.astype(np.float64), kind="stable")      # stable: equal keys keep position order
        want += sorted((lo + order[:m]).tolist())
    got = wo.select_tokens(key, seg, ret, 0)
    assert got.tolist() == want
    # every segment keeps exactly its quota: uniform temporal coverage
    for lo in range(0, T_a, seg):
        n = min(seg, T_a - lo)
        assert ((got >= lo) & (got < lo + n)).sum() == int(math.floor(r32 * n))
    # the global variant spends the same budget on the best positions of the whole head
    glob = wo.select_tokens(key, seg, ret, 1)
    order = np.argsort(-key.astype(np.float64), kind="stable")
    assert glob.tolist() == sorted(order[:total].tolist())
    assert len(glob) == len(got) == total
    assert key[glob].astype(np.float64).sum() >= key[got].astype(np.float64).sum() - 1e-9


def test_select_tokens_rejects_bad_arguments():
    with pytest.raises(wo.OracleError):
        wo.select_tokens([0.1, 0.2], 0, 0.5)
    with pytest.raises(wo.OracleError):
        wo.select_tokens([0.1, 0.2], 2, 1.5)


# ---------------------------------------------------------------- placement end to end
def _workload():
    w = tiny_custom(n_layers=2, n_q_heads=6, n_kv_heads=3, head_dim=64, n_text=7, audio_lens=(130,), chunk=16, budget=0.3,
                    roles=[[A, F, F], [T, F, A]], n_steps=3)
    w.n_prefill_queries = 4
    return w


@pytest.mark.parametrize("variant", [0, 1])
def test_token_placement_against_numpy(variant):
    w = _workload()
    syn = Synth(w, seed=4)
    o = make_oracle(w)
    seg = 25
    ret = np.array([[1.0, 0.3, 0.62], [0.5, 0.0, 1.0]], np.float32)       # per (layer, KV-head); only fixed heads use theirs
    scale = 1 / math.sqrt(w.head_dim)
    pre = {}
    for l in range(2):
        p = syn.prefill(0, l)
        kb, vb, qt = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_text"])
        o.place_prefill_tokens(0, l, kb, vb, p["audio_begin"], p["audio_end"], qt, ret[l], seg, variant)
        pre[l] = (bf16_bits_to_f64(kb), bf16_bits_to_f64(vb), qt, p["audio_begin"], p["audio_end"])
    kept = {}
    for l in range(2):
        K, V, qt, ab, ae = pre[l]
        for h in range(3):
            if w.roles[l, h] != F:
                assert o.fixed_tokens(0, l, h) is None
                continue
            want = np.zeros(ae - ab)
            for qi in range(4):
                for r in range(2):
                    _, prob = dense_attention(bf16_bits_to_f64(qt[qi, h * 2 + r]), K[:, h], V[:, h], scale)
                    want += prob[ab:ae]
            got = o.token_scores(0, l, h)
            assert np.abs(got - want).max() < 1e-13
            # the kept set is the per-segment (or global) top of that score, with this head's own retention
            m_tot, exp = 0, []
            k32 = want.astype(np.float32).astype(np.float64)
            for lo in range(0, ae - ab, seg):
                n = min(seg, ae - ab - lo)
                m = int(math.floor(float(ret[l, h]) * n)); m_tot += m
                exp += sorted((lo + np.argsort(-k32[lo:lo + n], kind="stable")[:m]).tolist())
            if variant == 1:
                exp = sorted(np.argsort(-k32, kind="stable")[:m_tot].tolist())
            kept[(l, h)] = o.fixed_tokens(0, l, h)
            assert kept[(l, h)].tolist() == exp
    assert len(kept[(1, 1)]) == 0 and len(kept[(0, 1)]) == 5 * 7 + 1     # floor(.3*25)=7 per segment, floor(.3*5)=1 in the tail
    # decode: a compressed fixed head attends to [text so far | its kept positions] and nothing else
    dec = {l: syn.decode(0, l) for l in range(2)}
    extra = {l: ([], []) for l in range(2)}
    for t in range(w.n_steps):
        o.step_begin([0])
        for l in range(2):
            q, kn, vn = (bf16_bits(dec[l][n][t]) for n in ("q", "k_new", "v_new"))
            out = o.decode_layer(l, q[None], kn[None], vn[None])
            extra[l][0].append(bf16_bits_to_f64(kn)); extra[l][1].append(bf16_bits_to_f64(vn))
            K, V, _, ab, ae = pre[l]
            text = [i for i in range(K.shape[0]) if not (ab <= i < ae)]
            for h in range(3):
                if w.roles[l, h] != F:
                    continue
                rows = text
                Kh = np.concatenate([K[rows, h], np.stack([x[h] for x in extra[l][0]]), K[ab:ae, h][kept[(l, h)]]])
                Vh = np.concatenate([V[rows, h], np.stack([x[h] for x in extra[l][1]]), V[ab:ae, h][kept[(l, h)]]])
                for r in range(2):
                    ref, _ = dense_attention(bf16_bits_to_f64(q[h * 2 + r]), Kh, Vh, scale)
                    assert np.abs(out[0, h * 2 + r] - ref).max() < 1e-12
        o.step_end()


def test_full_retention_equals_dense_attention_and_setter_round_trip():
    """retention 1 keeps every position: the fixed head then equals plain attention over the whole prefix."""
    w = _workload()
    syn = Synth(w, seed=5)
    o = make_oracle(w)
    pre = {}
    for l in range(2):
        p = syn.prefill(0, l)
        kb, vb, qt = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_text"])
        o.place_prefill_tokens(0, l, kb, vb, p["audio_begin"], p["audio_end"], qt, np.ones(3, np.float32), 25, 0)
        pre[l] = (bf16_bits_to_f64(kb), bf16_bits_to_f64(vb), p["audio_begin"], p["audio_end"])
    assert o.fixed_tokens(0, 0, 1).tolist() == list(range(130))
    q = bf16_bits(syn.decode(0, 0)["q"])[0]
    K, V, ab, ae = pre[0]
    scale = 1 / math.sqrt(w.head_dim)
    order = [i for i in range(K.shape[0]) if not (ab <= i < ae)] + list(range(ab, ae))
    q1 = bf16_bits(syn.decode(0, 1)["q"])[0]
    o.step_begin([0]); out = o.decode_layer(0, q[None]); o.decode_layer(1, q1[None]); o.step_end()
    for hq in (2, 3):                                                    # the q-heads of fixed KV-head 1
        ref, _ = dense_attention(bf16_bits_to_f64(q[hq]), K[order, 1], V[order, 1], scale)
        assert np.abs(out[0, hq] - ref).max() < 1e-12
    o.set_fixed_tokens(0, 0, 1, [3, 9, 77])
    assert o.fixed_tokens(0, 0, 1).tolist() == [3, 9, 77]
    p_row, _ = o.attention_row(0, 0, 2, q[2])
    T_t = o.dims(0)[1]
    assert sorted(np.nonzero(p_row[T_t:])[0].tolist()) == [3, 9, 77]
    assert abs(p_row.sum() - 1.0) < 1e-12


# ---------------------------------------------------------------- tidal heads with a token-granular base (residency 2)
def _lag_workload():
    w = tiny_custom(n_layers=2, n_q_heads=6, n_kv_heads=3, head_dim=64, n_text=6, audio_lens=(210,), chunk=25, budget=0.3,
                    roles=[[A, T, F], [T, T, A]], n_steps=6, topk=2, region=25, jump_every=2)
    w.n_prefill_queries = 3
    return w


@pytest.mark.parametrize("variant", [0, 1])
def test_token_base_tidal_heads_against_numpy(variant):
    """Residency 2: no segment is permanent as a whole; a tidal head sees [text | its kept positions | every position of the
    segments in its layer's dynamic slots].  Checked against numpy attention over exactly that key set, with the table
    advanced by the (separately pinned) lag update; retention 0 leaves a head with the fetched segments only, retention 1
    makes it plain dense attention."""
    w = _lag_workload()
    syn = Synth(w, seed=11)
    o = make_oracle(w, score_scope=1, residency=2, evict_lag=1)
    seg = w.chunk
    ret = np.array([[1.0, 0.3, 0.5], [0.0, 1.0, 1.0]], np.float32)
    scale = 1 / math.sqrt(w.head_dim)
    pre = {}
    with pytest.raises(wo.OracleError):                     # the chunk-granular placement has no base to offer here
        p = syn.prefill(0, 0)
        o.place_prefill(0, 0, bf16_bits(p["k"]), bf16_bits(p["v"]), p["audio_begin"], p["audio_end"], bf16_bits(p["q_text"]))
    for l in range(2):
        p = syn.prefill(0, l)
        kb, vb, qt = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_text"])
        o.place_prefill_tokens(0, l, kb, vb, p["audio_begin"], p["audio_end"], qt, ret[l], seg, variant)
        pre[l] = (bf16_bits_to_f64(kb), bf16_bits_to_f64(vb), qt, p["audio_begin"], p["audio_end"])
    T_a, T_t, C, S = o.dims(0)
    assert (C, S, o.base_slots(0)) == (9, 2 * 2 * 2, 0)      # D = 2*topk*(delta+1) dynamic slots, no permanent ones
    kept = {}
    for l in range(2):
        K, V, qt, ab, ae = pre[l]
        tab, _ = o.residency(0, l)
        assert (tab == -1).all()                              # nothing fetched yet
        for h in range(3):
            if w.roles[l, h] == A:
                continue
            want = np.zeros(T_a)
            for qi in range(3):
                for r in range(2):
                    _, prob = dense_attention(bf16_bits_to_f64(qt[qi, h * 2 + r]), K[:, h], V[:, h], scale)
                    want += prob[ab:ae]
            k32 = want.astype(np.float32).astype(np.float64)
            exp, m_tot = [], 0
            for lo in range(0, T_a, seg):
                n = min(seg, T_a - lo)
                m = int(math.floor(float(ret[l, h]) * n)); m_tot += m
                exp += sorted((lo + np.argsort(-k32[lo:lo + n], kind="stable")[:m]).tolist())
            if variant == 1:                      # the same budget spent on the best positions of the whole head
                exp = sorted(np.argsort(-k32, kind="stable")[:m_tot].tolist())
            kept[(l, h)] = o.fixed_tokens(0, l, h)
            assert kept[(l, h)].tolist() == exp
    assert len(kept[(1, 0)]) == 0 and len(kept[(1, 1)]) == T_a
    dec = {l: syn.decode(0, l) for l in range(2)}
    extra = {l: ([], []) for l in range(2)}
    seen_fetch = False
    for t in range(w.n_steps):
        tabs = {l: o.residency(0, l)[0] for l in range(2)}    # what attention of this step sees
        o.step_begin([0])
        for l in range(2):
            q, kn, vn = (bf16_bits(dec[l][n][t]) for n in ("q", "k_new", "v_new"))
            out = o.decode_layer(l, q[None], kn[None], vn[None])
            extra[l][0].append(bf16_bits_to_f64(kn)); extra[l][1].append(bf16_bits_to_f64(vn))
            K, V, _, ab, ae = pre[l]
            text = [i for i in range(K.shape[0]) if not (ab <= i < ae)]
            for h in range(3):
                if w.roles[l, h] == A:
                    continue
                vis = set(kept[(l, h)].tolist())
                if w.roles[l, h] == T:
                    for c in tabs[l]:
                        if c >= 0:
                            vis |= set(range(c * seg, min((c + 1) * seg, T_a)))
                            seen_fetch = True
                rows = sorted(vis)
                Kh = np.concatenate([K[text, h], np.stack([x[h] for x in extra[l][0]]), K[ab:ae, h][rows]])
                Vh = np.concatenate([V[text, h], np.stack([x[h] for x in extra[l][1]]), V[ab:ae, h][rows]])
                for r in range(2):
                    ref, _ = dense_attention(bf16_bits_to_f64(q[h * 2 + r]), Kh, Vh, scale)
                    assert np.abs(out[0, h * 2 + r] - ref).max() < 1e-12
        o.step_end()
    assert seen_fetch
    st = o.stats(0)
    assert st["misses"] > 0 and st["evictions"] > 0           # segments were fetched and released again
