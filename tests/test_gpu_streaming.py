"""Streaming audio on the GPU: a clip that grows between decode steps (wnw_append_audio), in lock-step with the oracle.

The harness places a prefix of the clip, then appends pieces between steps; everything the ordinary lock-step run
compares is compared here too (outputs, chunk scores, selections, tables and stamps, slot bytes), over chunks that
fill up, new chunks that enter tables through selection, a growing slot count, and fixed heads whose subset is final.
Needs a B200."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from helpers import make_oracle
from parity_harness import Lockstep
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, config1, tiny_custom
from workloads.synth import bf16_bits

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


class StreamingLockstep(Lockstep):
    """Lockstep whose sequences start with a prefix of their clip; append(b, n) hands over the next n positions."""

    def __init__(self, w, first, seed=0, mode=None, **kw):
        self.total = list(w.audio_lens)
        self.first = list(first)
        super().__init__(w, seed=seed, **kw)
        wnw.wnw_destroy(self.h)
        self.h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(self.total), w.text_capacity, w.chunk,
                                w.budget, w.roles, topk=w.topk, streaming_audio=1)
        self.pre = {}
        self.arrived = list(first)

    def prefill(self, check_slots=True):
        w = self.w
        for b in range(w.batch):
            for l in range(w.n_layers):
                self.pre[(b, l)] = self.syn.prefill(b, l)       # the whole clip's bits; only a prefix is placed
                self.dec[(b, l)] = self.syn.decode(b, l)        # decode inputs drawn for the whole clip, too
        real = w.audio_lens
        w.audio_lens = list(self.first)                          # what the harness believes the clip to be, for now
        orig = self.syn.prefill
        self.syn.prefill = lambda b, l: self._prefix(b, l)
        try:
            super().prefill(check_slots=check_slots)
        finally:
            self.syn.prefill = orig
        self.real = real

    def _prefix(self, b, l):
        p = dict(self.pre[(b, l)])
        n = self.w.n_text + self.first[b]
        p["k"], p["v"] = p["k"][:n].contiguous(), p["v"][:n].contiguous()
        p["n_tokens"], p["audio_end"] = n, n
        return p

    def append(self, b, n):
        w = self.w
        lo, hi = w.n_text + self.arrived[b], w.n_text + self.arrived[b] + n
        ks = [self.pre[(b, l)]["k"][lo:hi].contiguous() for l in range(w.n_layers)]
        vs = [self.pre[(b, l)]["v"][lo:hi].contiguous() for l in range(w.n_layers)]
        for l in range(w.n_layers):
            wnw.wnw_append_audio(self.h, b, l, ks[l].to(self.dev), vs[l].to(self.dev))
        torch.cuda.synchronize(self.dev)
        self.o.append_audio(b, np.stack([bf16_bits(x) for x in ks]), np.stack([bf16_bits(x) for x in vs]))
        for l in range(w.n_layers):                              # what check_slot_bytes compares the slots with
            kb, vb = self.kept[(b, l)]
            self.kept[(b, l)] = (np.concatenate([kb, bf16_bits(ks[l])]), np.concatenate([vb, bf16_bits(vs[l])]))
        self.arrived[b] += n
        w.audio_lens[b] = self.arrived[b]
        assert wnw.wnw_get_seq_dims(self.h, b) == self.o.dims(b)


def test_streaming_clip_in_lockstep_with_the_oracle():
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(400, 230), chunk=16, budget=0.3,
                    n_steps=12, roles=[[A, T, T, F], [T, F, A, T], [F, T, T, F]], region=16)
    ls = StreamingLockstep(w, first=(70, 33), seed=5)
    try:
        ls.prefill()
        plan = {1: (0, 5), 2: (1, 40), 4: (0, 150), 6: (1, 157), 7: (0, 175)}     # before step t: (sequence, positions)
        for t in range(12):
            if t in plan:
                ls.append(*plan[t])
            ls.decode_step(t, check_slots=True)
        ls.check_stats()
        assert ls.arrived == [400, 230]
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_streaming_with_replayed_steps_and_chained_layers():
    """Appends between replays: the captured step is captured again after every append (the work lists change)."""
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, n_text=5, audio_lens=(900,), chunk=64, budget=0.2,
                    n_steps=9, roles=[[A, T], [T, F]], region=64)
    ls = StreamingLockstep(w, first=(300,), seed=8)
    try:
        wnw.wnw_set_layer_dependency(ls.h, wnw.WNW_LAYERS_CHAINED)
        ls.prefill()
        for t in range(9):
            if t in (2, 5):
                ls.append(0, 300)
                ls._graph = None                                  # a new capture for the grown clip
            ls.decode_step(t, graph=True, check_slots=True)
        ls.check_stats()
    finally:
        ls.close()


def test_full_cache_mode_streams_too():
    """FULL mode stores every head in full: appended positions are visible to every head at once (numpy reference)."""
    from helpers import bf16_bits_to_f64, dense_attention
    n_q, n_kv, d, T0, T1 = 8, 2, 128, 100, 260
    gen = torch.Generator().manual_seed(3)
    k = torch.randn(T1, n_kv, d, generator=gen).to(torch.bfloat16)
    v = torch.randn(T1, n_kv, d, generator=gen).to(torch.bfloat16)
    q = (torch.randn(n_q, d, generator=gen) * 1.5).to(torch.bfloat16)
    h = wnw.wnw_create(1, n_q, n_kv, d, 1, T1, 16, 32, 0.2, np.zeros(n_kv, np.uint8), mode=wnw.WNW_MODE_FULL, streaming_audio=1)
    try:
        wnw.wnw_place_prefill(h, 0, 0, k[:T0].cuda(), v[:T0].cuda(), 0, T0)
        for upto in (T0, 117, T1):
            have = wnw.wnw_get_seq_dims(h, 0)[0]
            if upto > have:
                wnw.wnw_append_audio(h, 0, 0, k[have:upto].cuda(), v[have:upto].cuda())
            out = torch.zeros((1, n_q, d), dtype=torch.bfloat16, device="cuda")
            wnw.wnw_step_begin(h, [0])
            wnw.wnw_decode_layer_full(h, 0, q.cuda()[None], None, None, out)
            wnw.wnw_step_end(h)
            wnw.wnw_sync(h)
            got = out[0].float().cpu().numpy()
            for hq in range(n_q):
                ref, _ = dense_attention(bf16_bits_to_f64(bf16_bits(q))[hq], bf16_bits_to_f64(bf16_bits(k[:upto]))[:, hq // 4],
                                         bf16_bits_to_f64(bf16_bits(v[:upto]))[:, hq // 4], 1 / np.sqrt(d))
                assert np.abs(got[hq] - ref).max() <= 2e-2
    finally:
        wnw.wnw_destroy(h)


def test_append_audio_argument_and_state_errors():
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=4, audio_lens=(64,), chunk=16, n_steps=2,
                    roles=[[A, T], [T, F]])
    kv = torch.zeros((8, 2, 64), dtype=torch.bfloat16, device="cuda")
    def status(fn):
        with pytest.raises(wnw.WnwError) as e:
            fn()
        return e.value.status
    for streaming, expect in ((0, wnw.WNW_ERR_UNSUPPORTED),):
        ls = Lockstep(w, seed=1)
        try:
            ls.prefill()
            assert status(lambda: wnw.wnw_append_audio(ls.h, 0, 0, kv, kv)) == expect     # created without streaming_audio
        finally:
            ls.close()
    ls = StreamingLockstep(w, first=(40,), seed=1)
    try:
        ls.prefill()
        assert status(lambda: wnw.wnw_append_audio(ls.h, 0, 1, kv, kv)) == wnw.WNW_ERR_STATE        # layers in order
        wnw.wnw_append_audio(ls.h, 0, 0, kv, kv)
        assert status(lambda: wnw.wnw_step_begin(ls.h, [0])) == wnw.WNW_ERR_STATE                   # append unfinished
        assert status(lambda: wnw.wnw_append_audio(ls.h, 0, 1, kv[:4], kv[:4])) == wnw.WNW_ERR_STATE  # same count per layer
        wnw.wnw_append_audio(ls.h, 0, 1, kv, kv)
        big = torch.zeros((17, 2, 64), dtype=torch.bfloat16, device="cuda")
        assert status(lambda: wnw.wnw_append_audio(ls.h, 0, 0, big, big)) == wnw.WNW_ERR_CAPACITY   # 48 + 17 > 64
    finally:
        ls.close()
