"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element (needs a B200)."""
import numpy as np
import pytest
import torch

from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, config0, config1, config2, tiny_custom

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _run(w, n_steps=None, seed=0, append=True, recall_mode=0, check_slots=True):
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=seed, recall_mode=recall_mode)
    try:
        ls.prefill(check_slots=check_slots)
        for t in range(w.n_steps if n_steps is None else n_steps):
            ls.decode_step(t, append=append, check_slots=check_slots)
        ls.check_stats()
        return ls.near_ties, ls.max_out_err
    finally:
        ls.close()


def test_config0_all_steps():
    """Tiny single layer, 8q/4kv, d=64, roles {A,T,T,F}, 1024 audio tokens in 32 chunks, 16 steps, 20 % budget."""
    ties, err = _run(config0())
    assert ties == 0


@pytest.mark.parametrize("recall_mode", [0, 1])
def test_config0_recall_modes_agree(recall_mode):
    _run(config0(), recall_mode=recall_mode)


def test_config0_without_append():
    _run(config0(), append=False)


@pytest.mark.parametrize("audio_len,chunk,d,hq,hkv", [
    (100, 16, 64, 4, 2),      # ragged last chunk (100 = 6*16 + 4)
    (333, 32, 128, 8, 2),     # g = 4, several granules per chunk, ragged
    (257, 64, 128, 16, 2),    # g = 8
    (200, 16, 64, 32, 2),     # g = 16 (both row halves of the mma tile)
    (48, 16, 128, 2, 2),      # g = 1
    (1000, 256, 128, 8, 4),   # chunk spans many granules
    (3000 // 4, 50, 128, 8, 2),    # the paper's n_c = ceil(4 s * 12.5 tok/s) = 50: chunks stored padded to 64 rows
    (1500, 100, 128, 16, 2),       # n_c = ceil(4 s * 25 tok/s) = 100, g = 8
    (333, 25, 64, 4, 2),           # n_s = 25 tokens
    (77, 7, 64, 2, 2),             # smaller than a granule
])
def test_small_shapes(audio_len, chunk, d, hq, hkv):
    roles = [[A, T] + [F, T][: hkv - 2], [T, F] + [A, T][: hkv - 2], [A, F] + [T, T][: hkv - 2]]
    w = tiny_custom(n_layers=3, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, n_text=7, audio_lens=(audio_len,), chunk=chunk,
                    budget=0.34, n_steps=6, roles=roles, region=max(16, chunk // 2))
    _run(w, seed=11)


def test_ragged_batch_and_routing():
    """Three sequences of different lengths; layers without anchors route to the nearest anchor layer (both directions)."""
    roles = [[T, F], [A, T], [T, T], [T, F], [A, F], [F, F], [T, F]]
    w = tiny_custom(n_layers=7, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=9, audio_lens=(160, 75, 512), chunk=16,
                    budget=0.25, n_steps=8, roles=roles)
    _run(w, seed=4)


def test_budget_one_never_recalls_and_matches():
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=5, audio_lens=(130,), chunk=16, budget=1.0,
                    n_steps=4)
    _run(w, seed=2)


def test_no_audio_sequence():
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=20, audio_lens=(0,), chunk=16, n_steps=3)
    _run(w, seed=9)


def test_no_text_prefix():
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=0, audio_lens=(90,), chunk=16, n_steps=3)
    _run(w, seed=9)
    _run(w, seed=9, append=False)      # text region stays empty: tidal/fixed heads see audio only


def test_jumping_focus_turnover():
    """Focus jumps every 2 steps: every jump recalls chunks; slot bytes must equal the source KV after each recall."""
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640,), chunk=32, budget=0.2,
                    n_steps=12, roles=[[A, T, T, F], [T, A, F, T]], region=32, jump_every=2)
    _run(w, seed=6)


def test_graph_replay_matches_oracle():
    """A captured step replayed as a CUDA graph (side-stream selection and recall inside the graph) stays in
    lock-step with the oracle, also when eager steps are mixed in."""
    from parity_harness import Lockstep
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640, 300), chunk=32, budget=0.2,
                    n_steps=12, roles=[[A, T, T, F], [T, F, T, F], [A, T, F, T]], region=32, jump_every=3)
    ls = Lockstep(w, seed=8)
    try:
        ls.prefill()
        ls.decode_step(0, check_slots=True)                       # eager
        for t in range(1, 7):
            ls.decode_step(t, graph=True, check_slots=True)       # replay
        ls.decode_step(7, check_slots=True)                       # eager again
        for t in range(8, 12):
            ls.decode_step(t, graph=True, check_slots=True)
        ls.check_stats()
    finally:
        ls.close()


def test_config0_graph_replay_all_steps():
    from parity_harness import Lockstep
    ls = Lockstep(config0())
    try:
        ls.prefill()
        for t in range(16):
            ls.decode_step(t, graph=True, check_slots=True)
        ls.check_stats()
        assert ls.near_ties == 0
    finally:
        ls.close()


def test_config1_first_steps():
    """3B Voxtral-shaped stack (30 layers, 32q/8kv, d=128, 3000 audio tokens, chunk 64), first decode steps."""
    w = config1(n_steps=3)
    _run(w, check_slots=False)


def test_config2_first_steps():
    """3B Qwen-Omni-shaped stack (36 layers, 16q/2kv, d=128, 15000 audio tokens), routed layers, first decode steps."""
    w = config2(n_steps=2)
    _run(w, check_slots=False)


@pytest.mark.parametrize("n_q,audio_len,chunk,d,hq,hkv", [(5, 333, 32, 128, 8, 2), (17, 1000, 25, 64, 4, 2), (3, 77, 7, 64, 2, 2)])
def test_prefill_scores_summed_over_text_queries(n_q, audio_len, chunk, d, hq, hkv):
    """Prefill placement ranked by the attention of ALL text queries (one scoring pass per query, scores added), then
    decode steps on top of that placement."""
    roles = [[A, T], [T, F], [A, F]]
    w = tiny_custom(n_layers=3, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, n_text=7, audio_lens=(audio_len, audio_len // 2),
                    chunk=chunk, budget=0.3, n_steps=4, roles=roles, region=max(16, chunk))
    w.n_prefill_queries = n_q
    _run(w, seed=13)


def test_prefill_scores_summed_over_text_queries_config1_shape():
    w = config1(n_steps=2)
    w.n_layers = 4; w.roles = w.roles[:4]
    w.n_prefill_queries = 8
    _run(w, check_slots=False)


@pytest.mark.parametrize("residency", [0, 1])
def test_short_heads_packed_into_shared_ctas(residency):
    """Several short heads served by one CTA whose copy pipeline runs from one head into the next: the cut of a captured
    step whose layers are issued together, at a small shape, under the hard budget and under the lag residency."""
    import paper_2608_22704_b200 as wnw
    roles = [[A, T, T, F, T, F, T, T], [T, F, T, F, A, T, T, F], [A, T, F, T, T, T, F, F]]
    w = tiny_custom(n_layers=3, n_q_heads=16, n_kv_heads=8, head_dim=128, n_text=9, audio_lens=(640, 300, 75), chunk=32,
                    budget=0.2, n_steps=8, roles=roles, region=32, jump_every=3)
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=8, residency=residency, evict_lag=2)
    try:
        wnw.wnw_set_layer_dependency(ls.h, wnw.WNW_LAYERS_BATCHED)
        ls.prefill()
        for t in range(8):
            ls.decode_step(t, graph=t >= 2, check_slots=True)
        ls.check_stats()
    finally:
        ls.close()
