"""GPU parity at the full sizes of the batched configurations, in the launch configuration the benchmark times
(captured step replayed as a CUDA graph).  The oracle follows a sample of the sequences; inputs are generated on the
device and the sampled sequences' bits are copied to the host for the oracle.  (Needs a B200.)"""
import numpy as np
import pytest
import torch

from workloads import config1, config3, config4

pytestmark = pytest.mark.gpu


def _run(w, oracle_seqs, n_steps, graph=True, layer_dependency=0):
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=0, gen_device="cuda:0", oracle_seqs=oracle_seqs)
    try:
        wnw.wnw_set_layer_dependency(ls.h, layer_dependency)
        ls.prefill(check_slots=False)
        for t in range(n_steps):
            ls.decode_step(t, graph=graph, check_slots=(t == n_steps - 1))
        return ls.near_ties
    finally:
        ls.close()


@pytest.mark.parametrize("layer_dependency", [0, 1])
def test_config3_batch32_ragged_sampled_sequences(layer_dependency):
    """Batched serving: config-1 shapes at batch 32, audio lengths U{2000..7500}; the oracle follows the shortest and
    the longest sequence through prefill placement and three decode steps.  Independent layers run as one-shot CTAs
    (mostly one per head); chained layers run as persistent CTAs over the host-balanced schedule."""
    w = config3(n_steps=3)
    lens = np.array(w.audio_lens)
    _run(w, oracle_seqs=sorted({int(lens.argmin()), int(lens.argmax())}), n_steps=3, layer_dependency=layer_dependency)


@pytest.mark.parametrize("budget,chunk", [(0.1, 16), (0.4, 256)])
def test_config4_recall_stress_corners(budget, chunk):
    """Recall stress: batch 8 x 7500 audio tokens, focus jumping every 4 steps; corners of the budget x chunk grid
    (469 chunks of 16 tokens / 30 chunks of 256 tokens).  Five steps cover one jump; the last step also checks that
    every resident slot holds the exact bytes of its chunk."""
    w = config4(budget=budget, chunk=chunk, n_steps=5)
    _run(w, oracle_seqs=[3], n_steps=5)
    _run(w, oracle_seqs=[5], n_steps=2, layer_dependency=2)


def test_config1_sixty_four_steps_graph_replay():
    """3B Voxtral-shaped stack, 64 of the 256 decode steps (a quarter of the clip: the focus leaves the prefill set, chunks
    are recalled and evicted in every layer), replayed as a CUDA graph with overlapping layer kernels; the oracle follows
    every step.  Counters (hits, misses, evictions, recalled bytes) must agree at the end."""
    from parity_harness import Lockstep
    w = config1(n_steps=64)
    ls = Lockstep(w, seed=0, gen_device="cuda:0")
    try:
        ls.prefill(check_slots=False)
        for t in range(64):
            ls.decode_step(t, graph=True, check_slots=(t % 16 == 15))
        ls.check_stats()
        assert ls.near_ties == 0
        st = ls.o.stats(0)
        assert st["misses"] > 100 and st["evictions"] > 100      # the sweep really exercises recall and eviction
    finally:
        ls.close()


@pytest.mark.parametrize("residency,seg,scope", [(0, 64, 0), (1, 50, 0), (1, 50, 1)])
def test_config2_graph_replay(residency, seg, scope):
    """3B Qwen-Omni-shaped stack at full size (36 layers, 16q/2kv, g = 8, 15000 audio tokens = a 10-minute clip, layers
    without anchors routed to the nearest anchor layer) under graph replay: the contract's chunk-64 hard budget, and the
    paper's form for this tokeniser rate (50-token segments, chunks of two, lag-3 release), per-layer and global scores."""
    from parity_harness import Lockstep
    from workloads import config2
    w = config2(n_steps=6)
    w.chunk = seg
    ls = Lockstep(w, seed=0, gen_device="cuda:0", residency=residency, evict_lag=3, score_scope=scope)
    try:
        ls.prefill(check_slots=False)
        for t in range(6):
            ls.decode_step(t, graph=t >= 1, check_slots=(t == 5))
        ls.check_stats()
    finally:
        ls.close()


def test_config3_batch32_segment_lag_sampled_sequences():
    """Batch 32 ragged in the paper's form (25-token segments, lag release): one CTA per head, recall inside the step."""
    w = config3(n_steps=3)
    w.chunk = 25
    lens = np.array(w.audio_lens)
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=0, gen_device="cuda:0", oracle_seqs=sorted({int(lens.argmin()), int(lens.argmax())}),
                  residency=1, evict_lag=3)
    try:
        ls.prefill(check_slots=False)
        for t in range(3):
            ls.decode_step(t, graph=True, check_slots=(t == 2))
    finally:
        ls.close()


@pytest.mark.parametrize("residency,seg,dependency", [(0, 64, 0), (1, 25, 0), (0, 64, 3)])
def test_config1_whole_decode_graph_replay(residency, seg, dependency):
    """The whole 256-step decode of the 4-minute clip (text 64 -> 320 tokens, one full sweep of the focus through the audio)
    under graph replay, the oracle following every step: the contract's form and the paper's form with one launch per
    layer, and the contract's form with all layers issued together (the benchmark's default)."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    w = config1(n_steps=256)
    w.chunk = seg
    ls = Lockstep(w, seed=0, gen_device="cuda:0", residency=residency, evict_lag=3)
    try:
        wnw.wnw_set_layer_dependency(ls.h, dependency)
        ls.prefill(check_slots=False)
        for t in range(256):
            ls.decode_step(t, graph=True, check_slots=(t % 64 == 63))
        ls.check_stats()
        assert ls.near_ties <= 2
        st = ls.o.stats(0)
        assert st["misses"] > 500 and st["evictions"] > 400
        assert wnw_text_len(ls) == w.n_text + 256
    finally:
        ls.close()


def wnw_text_len(ls):
    import paper_2608_22704_b200 as wnw
    return wnw.wnw_get_seq_dims(ls.h, 0)[1]


@pytest.mark.parametrize("variant", [0, 1])
def test_config1_token_compressed_fixed_heads(variant):
    """Config 1 with its fixed heads compressed token by token in the paper's geometry (segments of 25 tokens = 2 s at
    12.5 tokens/s; per-head retention from Eq. 1 with seeded importances, lambda = 0.18, so a head keeps 0 to 4 positions
    of every segment of its 3000 audio tokens), four text queries; 12 decode steps replayed as a CUDA graph."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    w = config1(n_steps=12)
    w.n_prefill_queries = 4
    s_tilde = np.random.RandomState(7).rand(w.n_layers * w.n_kv_heads)
    ret = wnw.wnw_retention_schedule(s_tilde, 0.18).reshape(w.n_layers, w.n_kv_heads)
    ls = Lockstep(w, seed=2, gen_device="cuda:0", token_retention=ret, token_seg=25, token_variant=variant)
    try:
        ls.prefill(check_slots=False)
        for t in range(12):
            ls.decode_step(t, graph=True, check_slots=(t == 11))
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_config1_paper_form_with_token_base():
    """Config 1 in the paper's full form: 25-token segments, chunks of two segments, scores summed over all anchor layers,
    lag-3 release, and a token-granular permanent base: every tidal and fixed head keeps its per-segment best positions
    (per-head retention from Eq. 1, seeded importances, lambda = 0.36), tidal tables start empty and fetch complements.
    24 decode steps replayed as a CUDA graph; counters must agree at the end."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    w = config1(n_steps=24)
    w.chunk = 25
    w.n_prefill_queries = 2
    s_tilde = np.random.RandomState(11).rand(w.n_layers * w.n_kv_heads)
    ret = wnw.wnw_retention_schedule(s_tilde, 0.36).reshape(w.n_layers, w.n_kv_heads)
    ls = Lockstep(w, seed=3, gen_device="cuda:0", score_scope=1, residency=2, evict_lag=3, token_retention=ret, token_seg=25)
    try:
        ls.prefill(check_slots=False)
        for t in range(24):
            ls.decode_step(t, graph=True, check_slots=(t % 8 == 7))
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
        st = wnw.wnw_get_stats(ls.h)
        assert st["misses"] > 0
    finally:
        ls.close()
