"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only).

Each test states which part of the method it pins (Method section: Eq. 2 score
aggregation, Dynamic Chunk Selection, Prefill Compression, Method Overview for
the three head roles).  The reference attention here is a separate numpy
softmax (tests/helpers.dense_attention), not the oracle's own code.
"""
import itertools
import math

import numpy as np
import pytest

from helpers import bf16_bits_to_f64, dense_attention, f32_to_bf16_bits, make_oracle, place_all
from oracle import wnw_oracle as wo
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, config0, config1, config2, tiny_custom
from workloads.synth import bf16_bits


def _split(kept, b, l, h):
    K, V, _, ab, ae = kept[(b, l)]
    idx_text = [i for i in range(K.shape[0]) if not (ab <= i < ae)]
    return K[idx_text, h], V[idx_text, h], K[ab:ae, h], V[ab:ae, h]


# ---------------------------------------------------------------- hand-computable attention (scale, sign, operand order)
def test_two_key_closed_form():
    """q=(2,0,0,0), keys (1,0,0,0) and 0, d=4 => logits (2*1)/sqrt(4)=1 and 0 => p = e/(1+e), 1/(1+e)."""
    roles = np.array([[ROLE_ANCHOR]], np.uint8)
    o = wo.Oracle(1, 1, 1, 4, 1, 4, 4, 1, 1, 1.0, roles)
    K = np.zeros((2, 1, 4), np.float32); K[0, 0, 0] = 1.0
    V = np.zeros((2, 1, 4), np.float32); V[0, 0] = [1, 2, 3, 4]; V[1, 0] = [-1, 0, 1, 8]
    q = np.array([[2, 0, 0, 0]], np.float32)
    # token 0 is text, token 1 is audio
    o.place_prefill(0, 0, f32_to_bf16_bits(K), f32_to_bf16_bits(V), 1, 2, f32_to_bf16_bits(q))
    p, out = o.attention_row(0, 0, 0, f32_to_bf16_bits(q))
    p0 = math.e / (1 + math.e)
    assert p == pytest.approx([p0, 1 - p0], abs=1e-15)
    assert out == pytest.approx(p0 * np.array([1, 2, 3, 4.0]) + (1 - p0) * np.array([-1, 0, 1, 8.0]), abs=1e-14)
    o.step_begin([0])
    out2 = o.decode_layer(0, f32_to_bf16_bits(q)[None])
    o.step_end()
    assert out2[0, 0] == pytest.approx(out, abs=1e-15)
    # Eq. 2: the audio entry of the softmax over text+audio
    assert o.chunk_scores(0, 0) == pytest.approx([1 - p0], abs=1e-15)


# ---------------------------------------------------------------- rows sum to one
def test_softmax_rows_sum_to_one():
    w = config0()
    syn = Synth(w)
    o = make_oracle(w)
    place_all(o, syn)
    q = bf16_bits(syn.decode(0, 0)["q"])
    for hq in range(w.n_q_heads):            # anchor, tidal and fixed heads
        p, _ = o.attention_row(0, 0, hq, q[3, hq])
        assert abs(p.sum() - 1.0) < 1e-12
        assert (p >= 0).all()


# ---------------------------------------------------------------- budget 1.0 == full attention, with appends
@pytest.mark.parametrize("audio_len", [100, 96, 7])
def test_budget_one_equals_dense_attention(audio_len):
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=5, audio_lens=(audio_len,), chunk=16,
                    budget=1.0, n_steps=4)
    syn = Synth(w, seed=3)
    o = make_oracle(w)
    kept = place_all(o, syn, keep=True)
    dec = {l: syn.decode(0, l) for l in range(w.n_layers)}
    text_extra = {l: ([], []) for l in range(w.n_layers)}
    scale = 1 / math.sqrt(w.head_dim)
    for t in range(w.n_steps):
        o.step_begin([0])
        for l in range(w.n_layers):
            q, kn, vn = (bf16_bits(dec[l][n][t]) for n in ("q", "k_new", "v_new"))
            out = o.decode_layer(l, q[None], kn[None], vn[None])
            text_extra[l][0].append(bf16_bits_to_f64(kn)); text_extra[l][1].append(bf16_bits_to_f64(vn))
            for hq in range(w.n_q_heads):
                h = hq // w.group
                tK, tV, aK, aV = _split(kept, 0, l, h)
                K = np.concatenate([tK, np.stack([x[h] for x in text_extra[l][0]]), aK])
                V = np.concatenate([tV, np.stack([x[h] for x in text_extra[l][1]]), aV])
                ref, _ = dense_attention(bf16_bits_to_f64(q[hq]), K, V, scale)
                assert np.abs(out[0, hq] - ref).max() < 1e-12
        o.step_end()
    # at 100 % nothing is ever evicted or recalled
    st = o.stats(0)
    assert st["misses"] == 0 and st["evictions"] == 0


# ---------------------------------------------------------------- chunk scores = anchor heads' audio attention mass
def test_chunk_scores_sum_to_audio_mass():
    w = config0()
    syn = Synth(w)
    o = make_oracle(w)
    place_all(o, syn)
    dec = syn.decode(0, 0)
    q = bf16_bits(dec["q"])
    T_a, T_t, C, S = o.dims(0)
    mass = 0.0
    per_chunk = np.zeros(C)
    for hq in range(w.n_q_heads):
        if w.roles[0, hq // w.group] == ROLE_ANCHOR:
            p, _ = o.attention_row(0, 0, hq, q[0, hq])
            mass += 1.0 - p[:T_t].sum()
            per_chunk += p[T_t:].reshape(C, w.chunk).sum(axis=1)
    o.step_begin([0]); o.decode_layer(0, q[0][None]); o.step_end()
    sc = o.chunk_scores(0, 0)
    assert abs(sc.sum() - mass) < 1e-12
    assert np.abs(sc - per_chunk).max() < 1e-13


def test_chunk_scores_without_text_sum_to_anchor_head_count():
    w = tiny_custom(n_layers=1, n_q_heads=8, n_kv_heads=4, n_text=0, audio_lens=(90,), chunk=16,
                    roles=[[ROLE_ANCHOR, ROLE_TIDAL, ROLE_ANCHOR, ROLE_FIXED]], n_steps=2)
    syn = Synth(w, seed=1)
    o = make_oracle(w)
    place_all(o, syn)
    q = bf16_bits(syn.decode(0, 0)["q"])
    o.step_begin([0]); o.decode_layer(0, q[0][None]); o.step_end()
    assert abs(o.chunk_scores(0, 0).sum() - 4.0) < 1e-12      # 2 anchor KV-heads x group 2


# ---------------------------------------------------------------- closed forms
def test_identical_keys_uniform_scores_and_tie_break():
    """All keys identical => p = 1/(T_t+T_a); config-0 shapes: score_sum[c] = 2*32/1056; ties => sel = [0,1,2]."""
    w = config0()
    n = w.n_text + 1024
    rng = np.random.RandomState(0)
    krow = f32_to_bf16_bits(rng.randn(w.head_dim).astype(np.float32))
    K = np.broadcast_to(krow, (n, w.n_kv_heads, w.head_dim)).copy()
    V = f32_to_bf16_bits(rng.randn(n, w.n_kv_heads, w.head_dim).astype(np.float32))
    q = f32_to_bf16_bits(rng.randn(w.n_q_heads, w.head_dim).astype(np.float32))
    o = make_oracle(w)
    o.place_prefill(0, 0, K, V, w.n_text, n, q)
    # prefill ranking ties everywhere: fixed head and tidal table take chunks 0..S-1 in order
    assert o.fixed_set(0, 0, 3).tolist() == list(range(6))
    sc_, st_ = o.residency(0, 0)
    assert sc_.tolist() == list(range(6)) and st_.tolist() == [-1, -2, -3, -4, -5, -6]
    o.step_begin([0]); out = o.decode_layer(0, q[None]); o.step_end()
    sc = o.chunk_scores(0, 0)
    assert np.abs(sc - 2 * 32 / 1056).max() < 1e-14
    assert abs(sc.sum() - 2 * 1024 / 1056) < 1e-12
    assert o.selected(0, 0).tolist() == [0, 1, 2]
    # uniform attention: anchor output = mean of V over all positions
    Vf = bf16_bits_to_f64(V)
    assert np.abs(out[0, 0] - Vf[:, 0].mean(axis=0)).max() < 1e-12
    # three hits on resident chunks 0,1,2: stamps s*k + (k-1-r) with s=0, k=3
    sc_, st_ = o.residency(0, 0)
    assert sc_.tolist() == list(range(6)) and st_.tolist() == [2, 1, 0, -4, -5, -6]


def test_one_hot_key():
    """One audio key 40 nats above the rest: its chunk takes all the anchor mass, output -> that V row."""
    w = tiny_custom(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=3, audio_lens=(80,), chunk=16,
                    roles=[[ROLE_ANCHOR, ROLE_TIDAL]], n_steps=1)
    d = w.head_dim
    n = w.n_text + 80
    K = np.zeros((n, 2, d), np.float32); V = np.random.RandomState(1).randn(n, 2, d).astype(np.float32)
    hot = w.n_text + 37                                   # audio position 37 -> chunk 2
    K[hot, :, 0] = 40.0 * math.sqrt(d) / 2.0
    q = np.zeros((4, d), np.float32); q[:, 0] = 2.0       # logit = 2 * 40 sqrt(d)/2 / sqrt(d) = 40
    o = make_oracle(w)
    o.place_prefill(0, 0, f32_to_bf16_bits(K), f32_to_bf16_bits(V), w.n_text, n, f32_to_bf16_bits(q))
    o.step_begin([0]); out = o.decode_layer(0, f32_to_bf16_bits(q)[None]); o.step_end()
    sc = o.chunk_scores(0, 0)
    assert abs(sc[2] - 2.0) < 1e-14 and abs(sc.sum() - 2.0) < 1e-13          # 2 anchor q-heads
    assert np.abs(out[0, 0] - bf16_bits_to_f64(f32_to_bf16_bits(V))[hot, 0]).max() < 1e-13
    assert o.selected(0, 0)[0] == 2


# ---------------------------------------------------------------- top-k against brute force
def _brute_rank(score, lens):
    key = (np.asarray(score, np.float32) / np.asarray(lens, np.float32)).astype(np.float32)
    return sorted(range(len(score)), key=lambda c: (-float(key[c]), c))


@pytest.mark.parametrize("seed", range(20))
def test_topk_full_sort(seed):
    rng = np.random.RandomState(seed)
    C = int(rng.randint(1, 60))
    score = rng.rand(C).astype(np.float32)
    if seed % 2:                                         # forced ties
        score = np.round(score * 4) / 4
    lens = np.full(C, 16, np.int32); lens[-1] = rng.randint(1, 17)
    for k in (1, 3, C, C + 5):
        assert wo.topk(score, lens, k).tolist() == _brute_rank(score, lens)[:k]


@pytest.mark.parametrize("seed", range(10))
def test_topk_all_subsets(seed):
    """For C <= 8: the selected set maximises the key sum over all C-choose-k subsets and is the
    lexicographically smallest such set when ties exist."""
    rng = np.random.RandomState(100 + seed)
    C = int(rng.randint(3, 9)); k = 3
    score = (np.round(rng.rand(C) * 3) / 3).astype(np.float32)
    lens = np.full(C, 8, np.int32)
    key = (score / lens).astype(np.float32)
    sel = wo.topk(score, lens, k)
    best = max(itertools.combinations(range(C), k), key=lambda s: (sum(float(key[c]) for c in s), [-c for c in s]))
    assert sorted(sel.tolist()) == list(best)
    assert all(key[sel[i]] >= key[sel[i + 1]] for i in range(k - 1))


def test_topk_ranks_by_mean_not_sum():
    """The short last chunk is ranked by its own mean (Dynamic Chunk Selection: mean over tau in c)."""
    score = np.array([0.30, 0.20, 0.10], np.float32)     # sums
    lens = np.array([16, 16, 4], np.int32)               # means: .01875, .0125, .025
    assert wo.topk(score, lens, 3).tolist() == [2, 0, 1]


# ---------------------------------------------------------------- sparse heads == dense attention with a mask from the table
def test_tidal_and_fixed_equal_masked_dense_attention():
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(150,), chunk=16,
                    budget=0.3, n_steps=5)
    syn = Synth(w, seed=5)
    o = make_oracle(w)
    kept = place_all(o, syn, keep=True)
    dec = {l: syn.decode(0, l) for l in range(w.n_layers)}
    scale = 1 / math.sqrt(w.head_dim)
    T_a, T_t0, C, S = o.dims(0)
    assert C == 10 and S == 3
    for t in range(w.n_steps):
        tables = {l: o.residency(0, l)[0].copy() for l in range(w.n_layers)}   # as of end of step t-1
        o.step_begin([0])
        for l in range(w.n_layers):
            q = bf16_bits(dec[l]["q"][t])
            out = o.decode_layer(l, q[None])
            for hq in range(w.n_q_heads):
                h = hq // w.group
                role = w.roles[l, h]
                tK, tV, aK, aV = _split(kept, 0, l, h)
                if role == ROLE_ANCHOR:
                    vis = np.ones(C, bool)
                elif role == ROLE_TIDAL:
                    vis = np.zeros(C, bool); vis[[c for c in tables[l] if c >= 0]] = True
                else:
                    vis = np.zeros(C, bool); vis[o.fixed_set(0, l, h)] = True
                mask = np.concatenate([np.ones(len(tK), bool), np.repeat(vis, w.chunk)[:T_a]])
                ref, _ = dense_attention(bf16_bits_to_f64(q[hq]), np.concatenate([tK, aK]), np.concatenate([tV, aV]), scale, mask)
                assert np.abs(out[0, hq] - ref).max() < 1e-12
        o.step_end()


def test_output_invariant_under_slot_permutation():
    w = config0()
    syn = Synth(w)
    q = bf16_bits(syn.decode(0, 0)["q"][5])
    outs = []
    for perm_seed in (None, 1):
        o = make_oracle(w); place_all(o, syn)
        sc, st = o.residency(0, 0)
        if perm_seed is not None:
            perm = np.random.RandomState(perm_seed).permutation(len(sc))
            o.set_residency(0, 0, sc[perm], st[perm])
        o.step_begin([0]); outs.append(o.decode_layer(0, q[None])); o.step_end()
    assert np.abs(outs[0] - outs[1]).max() < 1e-13


# ---------------------------------------------------------------- prefill placement
def test_prefill_sets_are_top_chunks_of_numpy_prefill_attention():
    """Fixed head: own top-S chunks by mean prefill mass; tidal table: top-S of the mass summed over the layer's
    tidal heads, rank r in slot r (Prefill Compression, chunk-level)."""
    w = config0()
    syn = Synth(w)
    o = make_oracle(w)
    kept = place_all(o, syn, keep=True)
    K, V, qlast, ab, ae = kept[(0, 0)]
    scale = 1 / math.sqrt(w.head_dim)
    T_a, T_t, C, S = o.dims(0)
    assert (C, S) == (32, 6)
    pre = np.zeros((w.n_kv_heads, C))
    for hq in range(w.n_q_heads):
        h = hq // w.group
        _, p = dense_attention(qlast[hq], K[:, h], V[:, h], scale)
        pre[h] += p[ab:ae].reshape(C, w.chunk).sum(axis=1)
    for h in range(w.n_kv_heads):
        if w.roles[0, h] != ROLE_ANCHOR:
            assert np.abs(o.prefill_scores(0, 0, h) - pre[h]).max() < 1e-13
    lens = np.full(C, w.chunk)
    assert o.fixed_set(0, 0, 3).tolist() == _brute_rank(pre[3], lens)[:S]
    sc, st = o.residency(0, 0)
    assert sc.tolist() == _brute_rank(pre[1] + pre[2], lens)[:S]
    assert st.tolist() == [-1 - r for r in range(S)]
    # the sink on audio positions 0-3 puts chunk 0 first for a sink-dominated prefill query
    assert sc[0] == 0 and o.fixed_set(0, 0, 3)[0] == 0


@pytest.mark.parametrize("mk,expect", [(config0, (32, 6)), (config1, (47, 9)), (config2, (235, 47))])
def test_slot_counts_follow_floor_of_budget(mk, expect):
    """20 % of 32 chunks = 6 resident chunks (the tiny configuration's statement); floor elsewhere too."""
    w = mk()
    C = w.n_chunks(0)
    S = max(1, int(math.floor(float(np.float32(w.budget)) * C + 1e-6)))
    assert (C, S) == expect


# ---------------------------------------------------------------- routing
def test_score_routing_nearest_anchor_layer():
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    roles = np.array([[T, F], [A, T], [T, T], [T, F], [A, F], [F, F], [T, F]], np.uint8)
    o = wo.Oracle(7, 2, 2, 8, 1, 8, 8, 4, 1, 0.5, roles)
    # layer 0 -> 1; 1 -> itself; 2 -> 1; 3 -> 4; 4 has no tidal head; 5 none; 6 -> 4
    assert [o.score_source(l) for l in range(7)] == [1, 1, 1, 4, -1, -1, 4]
    roles2 = np.array([[A, F], [T, F], [T, F], [T, F], [A, F]], np.uint8)
    o2 = wo.Oracle(5, 2, 2, 8, 1, 8, 8, 4, 1, 0.5, roles2)
    assert [o2.score_source(l) for l in range(5)] == [-1, 0, 0, 4, -1]     # layer 2 is tied: lower layer wins


def test_routed_layer_uses_source_layers_scores_of_same_step():
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    w = tiny_custom(n_layers=3, n_q_heads=4, n_kv_heads=2, n_text=4, audio_lens=(128,), chunk=16, budget=0.5,
                    roles=[[T, F], [A, T], [T, T]], n_steps=3)
    syn = Synth(w, seed=2)
    o = make_oracle(w); place_all(o, syn)
    dec = {l: syn.decode(0, l) for l in range(3)}
    for t in range(3):
        o.step_begin([0])
        for l in range(3):
            o.decode_layer(l, bf16_bits(dec[l]["q"][t])[None])
        o.step_end()
        sc = o.chunk_scores(0, 1)
        want = _brute_rank(sc.astype(np.float32), np.full(8, 16))[:3]
        for l in range(3):
            assert o.selected(0, l).tolist() == want
            assert set(want) <= set(o.residency(0, l)[0].tolist())


# ---------------------------------------------------------------- selection takes effect one step later
def test_selection_used_from_next_step():
    w = config0()
    syn = Synth(w)
    o = make_oracle(w); place_all(o, syn)
    dec = syn.decode(0, 0)
    before = o.residency(0, 0)[0].copy()
    q8 = bf16_bits(dec["q"][8])
    # tidal q-head 2 sees exactly the chunks of the prefill table at step 0, whatever gets selected in that step
    p, _ = o.attention_row(0, 0, 2, q8[2])
    T_a, T_t, C, S = o.dims(0)
    seen = set(np.nonzero(p[T_t:].reshape(C, w.chunk).sum(axis=1))[0].tolist())
    assert seen == set(before.tolist())
    o.step_begin([0]); o.decode_layer(0, q8[None]); o.step_end()
    after = o.residency(0, 0)[0]
    sel = o.selected(0, 0)
    assert set(sel.tolist()) <= set(after.tolist())
    assert set(after.tolist()) != set(before.tolist())          # the drifting focus (step 8 of 16) is not in the prefill set
    p2, _ = o.attention_row(0, 0, 2, q8[2])
    seen2 = set(np.nonzero(p2[T_t:].reshape(C, w.chunk).sum(axis=1))[0].tolist())
    assert seen2 == set(after.tolist())


# ---------------------------------------------------------------- chunk geometry constants printed in the paper
def test_paper_chunk_geometry_constants():
    """W_c = 4 s, W_s = 2 s: 12.5 tok/s gives n_c = 50, n_s = 25; 25 tok/s gives 100 and 50 ("Chunk Structure")."""
    from workloads import paper_chunk_geometry
    assert paper_chunk_geometry(4, 2, 12.5) == (50, 25)
    assert paper_chunk_geometry(4, 2, 25) == (100, 50)


def test_oracle_accepts_the_papers_chunk_size():
    """Chunks of 50 tokens (not a multiple of anything convenient): budget 1.0 still equals dense attention and the
    chunk scores still sum to the anchor audio mass."""
    w = tiny_custom(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=3, audio_lens=(230,), chunk=50, budget=1.0,
                    roles=[[ROLE_ANCHOR, ROLE_TIDAL]], n_steps=1)
    syn = Synth(w, seed=4)
    o = make_oracle(w)
    kept = place_all(o, syn, keep=True)
    assert o.dims(0)[2:] == (5, 5)
    q = bf16_bits(syn.decode(0, 0)["q"][0])
    mass = 0.0
    for hq in (0, 1):
        p, _ = o.attention_row(0, 0, hq, q[hq])
        mass += p[3:].sum()
    o.step_begin([0]); out = o.decode_layer(0, q[None]); o.step_end()
    assert abs(o.chunk_scores(0, 0).sum() - mass) < 1e-12
    K, V, _, ab, ae = kept[(0, 0)]
    ref, _ = dense_attention(bf16_bits_to_f64(q[2]), K[:, 1], V[:, 1], 1 / math.sqrt(64))
    assert np.abs(out[0, 2] - ref).max() < 1e-12


# ---------------------------------------------------------------- global aggregation (Eq. 2 as printed)
def test_global_scope_sums_all_anchor_layers_and_shares_one_selection():
    """Score scope GLOBAL: every tidal layer selects from the sum of all anchor layers' chunk scores of the step."""
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    w = tiny_custom(n_layers=4, n_q_heads=4, n_kv_heads=2, n_text=4, audio_lens=(160,), chunk=16, budget=0.4,
                    roles=[[A, T], [T, F], [A, T], [T, T]], n_steps=3)
    syn = Synth(w, seed=7)
    o = make_oracle(w, score_scope=1); place_all(o, syn)
    dec = {l: syn.decode(0, l) for l in range(4)}
    for t in range(3):
        o.step_begin([0])
        for l in range(4):
            o.decode_layer(l, bf16_bits(dec[l]["q"][t])[None])
        o.step_end()
        glob = o.chunk_scores(0, 0) + o.chunk_scores(0, 2)
        want = _brute_rank(glob.astype(np.float32), np.full(10, 16))[:3]
        for l in range(4):
            assert o.selected(0, l).tolist() == want
    # per-layer scope on the same inputs routes layer 1 to layer 0 and layer 3 to layer 2 instead
    o2 = make_oracle(w, score_scope=0); place_all(o2, syn)
    o2.step_begin([0])
    for l in range(4):
        o2.decode_layer(l, bf16_bits(dec[l]["q"][0])[None])
    o2.step_end()
    assert o2.selected(0, 3).tolist() == _brute_rank(o2.chunk_scores(0, 2).astype(np.float32), np.full(10, 16))[:3]


def test_segment_lag_residency_end_to_end():
    """Residency SEGMENT_LAG (Chunk Structure + Dynamic Chunk Selection as printed): the paper's n_s = 25-token segments,
    chunks of two segments; the prefill segments stay for good; a fetched segment is dropped after delta unselected
    steps.  Checked through the whole oracle: dims, permanent base, selection from the overlapping-chunk means, the
    dynamic set against the window model, and tidal attention against dense attention masked by the table."""
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    delta, k = 2, 2
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(610,), chunk=25, budget=0.2,
                    roles=[[A, T], [T, F]], n_steps=12, topk=k, region=25, jump_every=3)
    syn = Synth(w, seed=13)
    o = make_oracle(w, residency=1, evict_lag=delta)
    kept = place_all(o, syn, keep=True)
    T_a, T_t0, C, S = o.dims(0)
    s_base = o.base_slots(0)
    assert C == 25 and s_base == 5 and S == s_base + 2 * k * (delta + 1)      # 610 tokens = 24 segments of 25 + one of 10
    lens = np.array([25] * 24 + [10])
    base = {l: o.residency(0, l)[0][:s_base].copy() for l in range(2)}
    assert all((o.residency(0, l)[0][s_base:] == -1).all() for l in range(2))
    assert len(o.fixed_set(0, 1, 1)) == s_base                                 # fixed heads keep the base amount only
    dec = {l: syn.decode(0, l) for l in range(2)}
    scale = 1 / math.sqrt(w.head_dim)
    history = {0: [], 1: []}
    moved = 0
    for t in range(w.n_steps):
        tables = {l: o.residency(0, l)[0].copy() for l in range(2)}
        o.step_begin([0])
        for l in range(2):
            q = bf16_bits(dec[l]["q"][t])
            out = o.decode_layer(l, q[None])
            h = 1 if l == 0 else 0                                             # the tidal head of the layer
            tK, tV, aK, aV = _split(kept, 0, l, h)
            vis = np.zeros(C, bool); vis[[c for c in tables[l] if c >= 0]] = True
            mask = np.concatenate([np.ones(len(tK), bool), np.repeat(vis, w.chunk)[:T_a]])
            for hq in range(h * 2, h * 2 + 2):
                ref, _ = dense_attention(bf16_bits_to_f64(q[hq]), np.concatenate([tK, aK]), np.concatenate([tV, aV]), scale, mask)
                assert np.abs(out[0, hq] - ref).max() < 1e-12
        o.step_end()
        sums = o.chunk_scores(0, 0).astype(np.float32)                         # layer 1 routes to layer 0
        keys = (sums[:-1] + sums[1:]) / (lens[:-1] + lens[1:]).astype(np.float32)
        want_chunks = sorted(range(C - 1), key=lambda j: (-float(keys[j]), j))[:k]
        for l in range(2):
            assert o.selected(0, l).tolist() == want_chunks
            segs = set()
            for j in want_chunks:
                segs |= {j, j + 1}
            history[l].append(segs)
            tab = o.residency(0, l)[0]
            assert tab[:s_base].tolist() == base[l].tolist()
            window = set().union(*history[l][-delta:]) - set(base[l].tolist())
            assert set(int(x) for x in tab[s_base:] if x >= 0) == window
            moved += len(window)
    assert moved > 0
    st = o.stats(0)
    assert st["misses"] > 0 and st["evictions"] > 0


def test_segment_lag_rejects_negative_lag():
    w = config0()
    with pytest.raises(wo.OracleError):
        make_oracle(w, residency=1, evict_lag=-1)


def test_prefill_scores_summed_over_text_queries():
    """"Prefill Compression": the prefill score aggregates the attention of ALL text queries.  With n_q queries the
    oracle's per-head chunk scores equal numpy dense attention summed over queries and q-heads, and (linearity) the sum
    of the scores the single-query form gives for each query alone; the placements are the top chunks of that sum."""
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    w = tiny_custom(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=6, audio_lens=(150,), chunk=16, budget=0.3,
                    roles=[[T, F]], n_steps=1)
    w.roles = np.array([[T, F]], np.uint8)
    w.n_prefill_queries = 5
    # a tidal head needs an anchor somewhere: add a second layer that has one
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=6, audio_lens=(150,), chunk=16, budget=0.3,
                    roles=[[T, F], [A, F]], n_steps=1)
    w.n_prefill_queries = 5
    syn = Synth(w, seed=9)
    p = syn.prefill(0, 0)
    kb, vb, qt = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_text"])
    assert qt.shape == (5, 4, 64)
    o = make_oracle(w)
    o.place_prefill(0, 0, kb, vb, p["audio_begin"], p["audio_end"], qt)
    scale = 1 / math.sqrt(w.head_dim)
    K, V = bf16_bits_to_f64(kb), bf16_bits_to_f64(vb)
    C = 10
    for h in range(2):
        want = np.zeros(C)
        for qi in range(5):
            for r in range(2):
                _, prob = dense_attention(bf16_bits_to_f64(qt[qi, h * 2 + r]), K[:, h], V[:, h], scale)
                aud = prob[p["audio_begin"]:p["audio_end"]]
                want += np.add.reduceat(aud, np.arange(0, 150, 16))
        got = o.prefill_scores(0, 0, h)
        assert np.abs(got - want).max() < 1e-12
        single = np.zeros(C)
        for qi in range(5):
            o1 = make_oracle(w)
            o1.place_prefill(0, 0, kb, vb, p["audio_begin"], p["audio_end"], qt[qi])
            single += o1.prefill_scores(0, 0, h)
            o1.close()
        assert np.abs(got - single).max() < 1e-12
    S = o.dims(0)[3]
    lens = np.array([16] * 9 + [6])
    assert o.fixed_set(0, 0, 1).tolist() == _brute_rank(o.prefill_scores(0, 0, 1).astype(np.float32), lens)[:S]
    assert o.residency(0, 0)[0].tolist() == _brute_rank(o.prefill_scores(0, 0, 0).astype(np.float32), lens)[:S]
