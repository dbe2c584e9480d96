"""GPU parity of the token-granular prefill compression of fixed heads (wnw_place_prefill_tokens) against the oracle:
per-position prefill scores, kept positions (bit-exact on the GPU's scores; equal to the oracle's own up to near-ties),
and the decode outputs of the compressed heads over several steps, eager and replayed.  Needs a B200."""
import math

import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, tiny_custom

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _workload(head_dim=128, n_kv=4, n_q=8, audio=(640, 300, 77), n_queries=3):
    w = tiny_custom(n_layers=3, n_q_heads=n_q, n_kv_heads=n_kv, head_dim=head_dim, n_text=9, audio_lens=audio, chunk=32, budget=0.5,
                    n_steps=8, roles=[[A, T, F, F][:n_kv], [T, F, T, F][:n_kv], [A, F, F, T][:n_kv]], region=32, jump_every=3)
    w.n_prefill_queries = n_queries
    return w


RET = np.array([[1.0, 1.0, 0.45, 0.2], [0.5, 0.0, 0.5, 0.33], [1.0, 0.04, 0.41, 0.9]], np.float32)


@pytest.mark.parametrize("variant", [0, 1])
def test_token_compressed_fixed_heads_follow_the_oracle(variant):
    """Three ragged sequences (640, 300, 77 audio tokens; segments of 25 leave a tail), per-head retention from 0
    (nothing kept: the head attends to text only) to 0.45 (several blocks with a ragged last one), both selection
    variants, eager and replayed steps."""
    from parity_harness import Lockstep
    w = _workload()
    ls = Lockstep(w, seed=21 + variant, token_retention=RET, token_seg=25, token_variant=variant)
    try:
        ls.prefill()
        for b in range(w.batch):
            T_a = w.audio_lens[b]
            for l in range(w.n_layers):
                for h in range(w.n_kv_heads):
                    if w.roles[l, h] != F:
                        continue
                    pos = wnw.wnw_get_fixed_tokens(ls.h, b, l, h)
                    want = sum(int(math.floor(float(RET[l, h]) * min(25, T_a - lo))) for lo in range(0, T_a, 25))
                    assert len(pos) == want and (np.diff(pos) > 0).all()
                    if variant == 0:                      # every segment keeps exactly its quota
                        for lo in range(0, T_a, 25):
                            n = min(25, T_a - lo)
                            assert ((pos >= lo) & (pos < lo + n)).sum() == int(math.floor(float(RET[l, h]) * n))
                    with pytest.raises(wnw.WnwError):      # a token-compacted head has no chunk set
                        wnw.wnw_get_fixed_set(ls.h, b, l, h)
        ls.decode_step(0, check_slots=True)
        for t in range(1, 5):
            ls.decode_step(t, graph=True, check_slots=True)
        ls.decode_step(5, check_slots=True)
        for t in range(6, 8):
            ls.decode_step(t, graph=True)
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_token_compression_d64_group4_single_query():
    """head_dim 64, four q-heads per KV-head, one text query, segments of 50 (the 25 tokens/s geometry)."""
    from parity_harness import Lockstep
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(1000,), chunk=16, budget=0.4,
                    n_steps=4, roles=[[A, F], [T, F]], region=16, jump_every=2)
    ret = np.array([[1.0, 0.37], [1.0, 0.1]], np.float32)
    ls = Lockstep(w, seed=3, token_retention=ret, token_seg=50)
    try:
        ls.prefill()
        for t in range(4):
            ls.decode_step(t, check_slots=True)
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_resident_token_count_and_r_gpu():
    """r_GPU accounting ("Metrics": audio KV tokens kept on the device): a compressed fixed head counts its kept positions."""
    from parity_harness import Lockstep
    w = _workload(audio=(640,))
    ls = Lockstep(w, seed=5, token_retention=RET, token_seg=25)
    try:
        ls.prefill()
        st = wnw.wnw_get_stats(ls.h)
        T_a = 640
        want = 0
        for l in range(w.n_layers):
            tab, _ = wnw.wnw_get_residency(ls.h, 0, l)
            for h in range(w.n_kv_heads):
                if w.roles[l, h] == A:
                    want += T_a
                elif w.roles[l, h] == T:
                    want += sum(min(32, T_a - int(c) * 32) for c in tab if c >= 0)
                else:
                    want += len(wnw.wnw_get_fixed_tokens(ls.h, 0, l, h))
        assert st["resident_audio_tokens"] == want
        assert st["full_audio_tokens"] == w.n_layers * w.n_kv_heads * T_a
    finally:
        ls.close()


def test_token_placement_argument_and_capacity_errors():
    w = _workload(audio=(640,))
    h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, 1, 640, w.text_capacity, w.chunk, 0.2, w.roles,
                       topk=w.topk)
    try:
        syn = Synth(w, seed=1)
        p = syn.prefill(0, 0)
        k, v, q = (p[n].cuda() for n in ("k", "v", "q_text"))
        args = (h, 0, 0, k, v, p["audio_begin"], p["audio_end"], q)
        with pytest.raises(wnw.WnwError) as e:      # 0.9 of 640 positions do not fit a store of 4 slots x 32 rows
            wnw.wnw_place_prefill_tokens(*args, [1, 1, 0.9, 0.1], 25)
        assert e.value.status == wnw.WNW_ERR_CAPACITY
        for bad in ([1, 1, 1.5, 0.1], [1, 1, -0.1, 0.1], [1, 1, float("nan"), 0.1]):
            with pytest.raises(wnw.WnwError) as e:
                wnw.wnw_place_prefill_tokens(*args, bad, 25)
            assert e.value.status == wnw.WNW_ERR_INVALID_ARG
        with pytest.raises(wnw.WnwError):
            wnw.wnw_place_prefill_tokens(*args, [1, 1, 0.1, 0.1], 0)
        with pytest.raises(wnw.WnwError):
            wnw.wnw_place_prefill_tokens(*args, [1, 1, 0.1, 0.1], 25, variant=2)
        # nothing was placed by the failed calls: a valid one still starts the sequence at layer 0
        wnw.wnw_place_prefill_tokens(*args, [1, 1, 0.15, 0.1], 25)
        wnw.wnw_sync(h)
        assert len(wnw.wnw_get_fixed_tokens(h, 0, 0, 2)) == 25 * 3 + 2      # floor(.15*25)=3 per segment, floor(.15*15)=2
        with pytest.raises(wnw.WnwError):            # scores are those of the most recent placement only
            wnw.wnw_get_token_scores(h, 0, 1, 1)
    finally:
        wnw.wnw_destroy(h)


def test_retention_schedule_on_the_host():
    r = wnw.wnw_retention_schedule([0.0, 0.1, 0.5, 1.0], 1.5)
    assert r.tolist() == [0.0, np.float32(0.1) * np.float32(1.5), 0.75, 1.0]
    with pytest.raises(wnw.WnwError):
        wnw.wnw_retention_schedule([0.5, 1.2], 1.0)


# ---------------------------------------------------------------- tidal heads with a token-granular permanent base
def _lag_workload(audio=(640, 300, 77), chunk=25, head_dim=128, n_steps=10):
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=head_dim, n_text=9, audio_lens=audio, chunk=chunk, budget=0.3,
                    n_steps=n_steps, roles=[[A, T, F, T], [T, F, T, F], [A, T, T, T]], region=chunk, jump_every=3, topk=2)
    w.n_prefill_queries = 3
    return w


RET_LAG = np.array([[1.0, 0.3, 0.45, 0.0], [0.5, 0.2, 0.08, 0.33], [1.0, 0.41, 0.25, 0.5]], np.float32)


@pytest.mark.parametrize("scope,variant", [(0, 0), (1, 0), (0, 1)])
def test_token_base_tidal_heads_follow_the_oracle(scope, variant):
    """Residency SEGMENT_LAG_TOKEN_BASE: every tidal head keeps its own per-segment best positions for good (retention
    0 to 0.5 per head), tables start empty, selected segments are fetched as complements (host mirror permuted) and
    released after the lag; per-layer and global score scope; per-segment quota and the global top-k variant (a base then
    holds a different number of positions in every segment); eager and replayed steps; slot bytes checked against the
    permuted source rows."""
    from parity_harness import Lockstep
    w = _lag_workload()
    ls = Lockstep(w, seed=31 + scope, score_scope=scope, residency=2, evict_lag=1, token_retention=RET_LAG, token_seg=25,
                  token_variant=variant)
    try:
        ls.prefill()
        for b in range(w.batch):
            assert wnw.wnw_get_base_slots(ls.h, b) == 0
            for l in range(w.n_layers):
                tab, _ = wnw.wnw_get_residency(ls.h, b, l)
                assert (tab == -1).all()
        ls.decode_step(0, check_slots=True)
        for t in range(1, 6):
            ls.decode_step(t, graph=True, check_slots=True)
        ls.decode_step(6, check_slots=True)
        for t in range(7, 10):
            ls.decode_step(t, graph=True, check_slots=(t == 9))
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
        st = wnw.wnw_get_stats(ls.h)
        assert st["misses"] > 0 and st["evictions"] > 0
        # r_GPU accounting: kept positions plus the complements of the fetched segments, per tidal head
        want = 0
        for b in range(w.batch):
            T_a = w.audio_lens[b]
            C = -(-T_a // 25)
            for l in range(w.n_layers):
                tab, _ = wnw.wnw_get_residency(ls.h, b, l)
                for h in range(w.n_kv_heads):
                    if w.roles[l, h] == A:
                        want += T_a
                        continue
                    kept = wnw.wnw_get_fixed_tokens(ls.h, b, l, h)
                    want += len(kept)
                    if w.roles[l, h] == T:
                        ks = set(kept.tolist())
                        for c in tab:
                            if c >= 0:
                                want += sum(1 for p in range(c * 25, min((c + 1) * 25, T_a)) if p not in ks)
        assert st["resident_audio_tokens"] == want
    finally:
        ls.close()


def test_token_base_chunk_of_64_and_d64():
    """Segments of 64 tokens (four granules per block), head_dim 64, a sequence whose last segment is short."""
    from parity_harness import Lockstep
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(1000, 130), chunk=64, budget=0.25,
                    n_steps=6, roles=[[A, T], [T, F]], region=64, jump_every=2, topk=3)
    ret = np.array([[1.0, 0.3], [0.17, 0.4]], np.float32)
    ls = Lockstep(w, seed=4, residency=2, evict_lag=2, token_retention=ret, token_seg=64)
    try:
        ls.prefill()
        for t in range(6):
            ls.decode_step(t, graph=(t % 2 == 1), check_slots=True)
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_token_base_placement_rules():
    w = _lag_workload(audio=(640,))
    h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, 1, 640, w.text_capacity, w.chunk, w.budget, w.roles,
                       topk=w.topk, residency=wnw.WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE, evict_lag=1)
    try:
        p = Synth(w, seed=1).prefill(0, 0)
        k, v, q = (p[n].cuda() for n in ("k", "v", "q_text"))
        with pytest.raises(wnw.WnwError) as e:       # the chunk-granular placement has no base to offer
            wnw.wnw_place_prefill(h, 0, 0, k, v, p["audio_begin"], p["audio_end"], q)
        assert e.value.status == wnw.WNW_ERR_STATE
        args = (h, 0, 0, k, v, p["audio_begin"], p["audio_end"], q, RET_LAG[0])
        with pytest.raises(wnw.WnwError) as e:       # the quota's segment is the storage segment
            wnw.wnw_place_prefill_tokens(*args, 50, 0)
        assert e.value.status == wnw.WNW_ERR_UNSUPPORTED
        wnw.wnw_place_prefill_tokens(*args, 25, 0)
        wnw.wnw_sync(h)
        assert len(wnw.wnw_get_fixed_tokens(h, 0, 0, 1)) == 25 * 7 + 4       # floor(.3*25)=7, tail floor(.3*15)=4
        assert len(wnw.wnw_get_fixed_tokens(h, 0, 0, 3)) == 0
    finally:
        wnw.wnw_destroy(h)
