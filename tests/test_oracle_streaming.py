"""Pins of the oracle's streaming-audio reading (CPU only): a clip that grows between decode steps.

The paper names streaming as the method's setting (Limitations section) without saying how a growing clip enters the
tiers; the reading the oracle takes is stated in its header.  What fixes it here is independent of the oracle's own
code: numpy dense attention over explicit position masks, the slot rule as a closed form, and the equivalence of
"arrived in pieces" with "placed whole" where the reading makes them equal."""
import math

import numpy as np

from helpers import bf16_bits_to_f64, dense_attention
from oracle.wnw_oracle import Oracle
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, tiny_custom
from workloads.synth import bf16_bits

A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _oracle(w, roles=None, max_audio=None):
    return Oracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, 1, max_audio or w.audio_lens[0], w.text_capacity, w.chunk,
                  w.topk, w.budget, w.roles if roles is None else roles)


class Clip:
    """The whole clip's bits per layer; placement takes a prefix of the audio, appends hand over the next positions."""

    def __init__(self, w, seed):
        self.w = w
        self.syn = Synth(w, seed=seed)
        self.pre = [self.syn.prefill(0, l) for l in range(w.n_layers)]
        self.k = [bf16_bits(p["k"]) for p in self.pre]
        self.v = [bf16_bits(p["v"]) for p in self.pre]
        self.q = [bf16_bits(p["q_last"]) for p in self.pre]
        self.dec = [self.syn.decode(0, l) for l in range(w.n_layers)]
        self.nt = w.n_text

    def place(self, o, n_audio):
        for l in range(self.w.n_layers):
            n = self.nt + n_audio
            o.place_prefill(0, l, self.k[l][:n], self.v[l][:n], self.nt, n, self.q[l])

    def append(self, o, lo, hi):
        k = np.stack([self.k[l][self.nt + lo:self.nt + hi] for l in range(self.w.n_layers)])
        v = np.stack([self.v[l][self.nt + lo:self.nt + hi] for l in range(self.w.n_layers)])
        o.append_audio(0, k, v)

    def step(self, o, t):
        """One decode step with appends of generated tokens; returns [layer] -> out [Hq, d]."""
        o.step_begin([0])
        outs = []
        for l in range(self.w.n_layers):
            d = self.dec[l]
            outs.append(o.decode_layer(l, bf16_bits(d["q"][t])[None], bf16_bits(d["k_new"][t])[None], bf16_bits(d["v_new"][t])[None])[0])
        o.step_end()
        return outs


def test_anchor_heads_arrival_in_pieces_equals_the_whole_clip():
    """All heads anchors: after the last piece has arrived the outputs are those of an oracle that was given the whole
    clip at once, bit for bit; while the clip is still growing they equal numpy attention over what has arrived."""
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(150,), chunk=16, n_steps=6)
    roles = np.zeros((2, 2), np.uint8)
    clip = Clip(w, seed=3)
    whole, grown = _oracle(w, roles), _oracle(w, roles)
    clip.place(whole, 150)
    clip.place(grown, 40)                       # 2.5 chunks: the short last chunk fills up first
    arrived = 40
    scale = 1 / math.sqrt(w.head_dim)
    for t, upto in enumerate((40, 47, 100, 150, 150, 150)):
        if upto > arrived:
            clip.append(grown, arrived, upto)
            arrived = upto
        assert grown.dims(0)[0] == arrived and grown.dims(0)[2] == -(-arrived // 16)
        og = clip.step(grown, t)
        ow = clip.step(whole, t)
        for l in range(w.n_layers):
            for hq in range(w.n_q_heads):
                h = hq // w.group
                n_txt = w.n_text + t + 1
                K = np.concatenate([bf16_bits_to_f64(clip.k[l][:w.n_text, h]),
                                    bf16_bits_to_f64(np.stack([bf16_bits(clip.dec[l]["k_new"][s][h]) for s in range(t + 1)])),
                                    bf16_bits_to_f64(clip.k[l][w.n_text:w.n_text + arrived, h])])
                V = np.concatenate([bf16_bits_to_f64(clip.v[l][:w.n_text, h]),
                                    bf16_bits_to_f64(np.stack([bf16_bits(clip.dec[l]["v_new"][s][h]) for s in range(t + 1)])),
                                    bf16_bits_to_f64(clip.v[l][w.n_text:w.n_text + arrived, h])])
                assert len(K) == n_txt + arrived
                ref, _ = dense_attention(bf16_bits_to_f64(bf16_bits(clip.dec[l]["q"][t])[hq]), K, V, scale)
                assert np.abs(og[l][hq] - ref).max() < 1e-12
            if arrived == 150:
                assert np.array_equal(og[l], ow[l])


def test_every_role_equals_dense_attention_over_an_explicit_position_mask():
    """Roles {anchor, tidal, tidal, fixed}: anchor heads see every arrived position; tidal heads the arrived positions of
    the chunks in the table as it stood before the step (a resident chunk that grew is seen grown, a new chunk is not seen
    until a selection brought it in); fixed heads their prefill chunks clipped to what had arrived at placement."""
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(200,), chunk=16, budget=0.3,
                    n_steps=7, roles=[[A, T, T, F], [T, F, A, T]], region=16)
    clip = Clip(w, seed=9)
    o = _oracle(w)
    T0 = 70                                   # 4 full chunks + one of 6 tokens
    clip.place(o, T0)
    arrived = T0
    scale = 1 / math.sqrt(w.head_dim)
    fixed_sets = {(l, h): o.fixed_set(0, l, h).copy() for l in range(2) for h in range(4) if w.roles[l, h] == F}
    saw_new_chunk_in_table = False
    for t, upto in enumerate((70, 75, 75, 130, 130, 200, 200)):
        if upto > arrived:
            before = {l: o.residency(0, l) for l in range(2)}
            clip.append(o, arrived, upto)
            arrived = upto
            T_a, _, C, S = o.dims(0)
            assert (T_a, C) == (arrived, -(-arrived // 16))
            assert S == max(1, int(math.floor(np.float32(0.3) * C + 1e-6)))      # the slot rule on the grown clip
            for l in range(2):                                                     # tables carry over, added slots are empty
                tab, stamp = o.residency(0, l)
                n_old = len(before[l][0])
                assert tab[:n_old].tolist() == before[l][0].tolist() and stamp[:n_old].tolist() == before[l][1].tolist()
                assert (tab[n_old:] == -1).all()
            for key, fs in fixed_sets.items():                                     # fixed sets are final
                assert o.fixed_set(0, *key).tolist() == fs.tolist()
        tables = {l: o.residency(0, l)[0].copy() for l in range(2)}
        C = o.dims(0)[2]
        outs = clip.step(o, t)
        scores = {l: o.chunk_scores(0, l) for l in range(2)}
        for l in range(2):
            assert len(scores[l]) == C                                             # new chunks are scored from their first step
            for hq in range(w.n_q_heads):
                h = hq // w.group
                role = w.roles[l, h]
                pos = np.zeros(arrived, bool)
                if role == A:
                    pos[:] = True
                elif role == T:
                    for c in tables[l]:
                        if c >= 0:
                            pos[c * 16:min((c + 1) * 16, arrived)] = True
                            saw_new_chunk_in_table |= c * 16 >= T0
                else:
                    for c in fixed_sets[(l, h)]:
                        pos[c * 16:min((c + 1) * 16, T0)] = True                   # never beyond what had arrived at placement
                K = np.concatenate([bf16_bits_to_f64(clip.k[l][:w.n_text, h]),
                                    bf16_bits_to_f64(np.stack([bf16_bits(clip.dec[l]["k_new"][s][h]) for s in range(t + 1)])),
                                    bf16_bits_to_f64(clip.k[l][w.n_text:w.n_text + arrived, h])])
                V = np.concatenate([bf16_bits_to_f64(clip.v[l][:w.n_text, h]),
                                    bf16_bits_to_f64(np.stack([bf16_bits(clip.dec[l]["v_new"][s][h]) for s in range(t + 1)])),
                                    bf16_bits_to_f64(clip.v[l][w.n_text:w.n_text + arrived, h])])
                mask = np.concatenate([np.ones(w.n_text + t + 1, bool), pos])
                ref, p = dense_attention(bf16_bits_to_f64(bf16_bits(clip.dec[l]["q"][t])[hq]), K, V, scale, mask)
                assert np.abs(outs[l][hq] - ref).max() < 1e-12, (t, l, hq, role)
        # chunk scores of an anchor layer: the anchor q-heads' softmax mass on every arrived chunk (Eq. 2 summed per chunk)
        for l in range(2):
            tot = 0.0
            for hq in range(w.n_q_heads):
                h = hq // w.group
                if w.roles[l, h] != A:
                    continue
                K = np.concatenate([bf16_bits_to_f64(clip.k[l][:w.n_text, h]),
                                    bf16_bits_to_f64(np.stack([bf16_bits(clip.dec[l]["k_new"][s][h]) for s in range(t + 1)])),
                                    bf16_bits_to_f64(clip.k[l][w.n_text:w.n_text + arrived, h])])
                _, p = dense_attention(bf16_bits_to_f64(bf16_bits(clip.dec[l]["q"][t])[hq]), K, K, scale)
                tot += p[w.n_text + t + 1:].sum()
            assert abs(scores[l].sum() - tot) < 1e-10
    assert saw_new_chunk_in_table          # the drifting focus did pull chunks that arrived after placement into a table


def test_append_is_refused_inside_a_step_and_beyond_capacity():
    w = tiny_custom(n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=64, n_text=3, audio_lens=(64,), chunk=16, n_steps=2,
                    roles=[[A, T]])
    clip = Clip(w, seed=1)
    o = _oracle(w)
    clip.place(o, 32)
    import pytest
    from oracle.wnw_oracle import OracleError
    o.step_begin([0])
    with pytest.raises(OracleError):
        clip.append(o, 32, 40)
    d = clip.dec[0]
    o.decode_layer(0, bf16_bits(d["q"][0])[None], None, None)
    o.step_end()
    clip.append(o, 32, 64)
    with pytest.raises(OracleError):        # the cache was created for 64 audio tokens
        o.append_audio(0, np.zeros((1, 1, 2, 64), np.uint16), np.zeros((1, 1, 2, 64), np.uint16))


def test_a_fixed_head_that_keeps_the_short_last_chunk_does_not_see_it_grow():
    """Budget 1.0: the fixed head keeps every chunk that existed at placement, the short last one included.  When that
    chunk fills up and new chunks follow, the fixed head still attends to exactly the positions that had arrived at
    placement, while the tidal head of the same layer (all of its chunks resident, new slots empty) sees the old chunks
    grown and the anchor head everything."""
    w = tiny_custom(n_layers=1, n_q_heads=3, n_kv_heads=3, head_dim=64, n_text=4, audio_lens=(100,), chunk=16, budget=1.0,
                    n_steps=3, roles=[[A, T, F]])
    clip = Clip(w, seed=4)
    o = _oracle(w)
    T0 = 37                                   # chunks 0, 1 full, chunk 2 holds 5 tokens
    clip.place(o, T0)
    assert sorted(o.fixed_set(0, 0, 2).tolist()) == [0, 1, 2]
    clip.append(o, T0, 100)
    tab = o.residency(0, 0)[0]
    assert sorted(tab[tab >= 0].tolist()) == [0, 1, 2] and o.dims(0)[3] == 7
    outs = clip.step(o, 0)
    scale = 1 / math.sqrt(w.head_dim)
    for h, upto in ((0, 100), (1, 48), (2, T0)):       # anchor: all; tidal: chunks 0-2 as they are now; fixed: as they were
        K = np.concatenate([bf16_bits_to_f64(clip.k[0][:w.n_text, h]), bf16_bits_to_f64(bf16_bits(clip.dec[0]["k_new"][0][h]))[None],
                            bf16_bits_to_f64(clip.k[0][w.n_text:w.n_text + upto, h])])
        V = np.concatenate([bf16_bits_to_f64(clip.v[0][:w.n_text, h]), bf16_bits_to_f64(bf16_bits(clip.dec[0]["v_new"][0][h]))[None],
                            bf16_bits_to_f64(clip.v[0][w.n_text:w.n_text + upto, h])])
        ref, _ = dense_attention(bf16_bits_to_f64(bf16_bits(clip.dec[0]["q"][0])[h]), K, V, scale)
        assert np.abs(outs[0][h] - ref).max() < 1e-12, h
