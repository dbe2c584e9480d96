"""GPU parity for SEGMENT_LAG residency ("Chunk Structure" and "Dynamic Chunk Selection" as printed): overlapping
two-segment chunks, permanent prefill base, fetched segments released after delta unselected steps (needs a B200)."""
import numpy as np
import pytest

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, config1, tiny_custom

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
LAG = wnw.WNW_RESIDENCY_SEGMENT_LAG


def _run(w, delta=3, seed=0, graph_from=None, scope=0, dependency=0, check_slots=True, n_steps=None):
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=seed, residency=LAG, evict_lag=delta, score_scope=scope)
    try:
        wnw.wnw_set_layer_dependency(ls.h, dependency)
        ls.prefill(check_slots=check_slots)
        s_base = [wnw.wnw_get_base_slots(ls.h, b) for b in range(w.batch)]
        base = {(b, l): wnw.wnw_get_residency(ls.h, b, l)[0][:s_base[b]].copy() for b in range(w.batch)
                for l in range(w.n_layers) if (w.roles[l] == T).any()}
        for t in range(w.n_steps if n_steps is None else n_steps):
            ls.decode_step(t, graph=graph_from is not None and t >= graph_from, check_slots=check_slots)
            for (b, l), want in base.items():       # what was placed at prefill stays
                assert np.array_equal(wnw.wnw_get_residency(ls.h, b, l)[0][:s_base[b]], want)
        ls.check_stats()
        return ls
    finally:
        ls.close()


@pytest.mark.parametrize("audio_len,seg,d,hq,hkv,delta,topk", [
    (610, 25, 64, 4, 2, 2, 2),       # the paper's n_s = 25 (12.5 tokens/s), ragged last segment
    (1500, 50, 128, 16, 2, 3, 3),    # n_s = 50 (25 tokens/s), g = 8, the paper's k = 3 and delta = 3
    (333, 16, 128, 8, 2, 1, 3),      # delta = 1
    (257, 32, 64, 8, 4, 0, 1),       # delta = 0: a fetched segment lives for one step
    (40, 25, 64, 2, 2, 3, 3),        # two segments: one chunk
    (20, 25, 64, 2, 2, 3, 3),        # one segment
])
def test_small_shapes_lag(audio_len, seg, d, hq, hkv, delta, topk):
    roles = [[A, T] + [F, T][: hkv - 2], [T, F] + [A, T][: hkv - 2], [A, F] + [T, T][: hkv - 2]]
    w = tiny_custom(n_layers=3, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, n_text=7, audio_lens=(audio_len,), chunk=seg,
                    budget=0.2, n_steps=10, roles=roles, region=max(16, seg), jump_every=3, topk=topk)
    _run(w, delta=delta, seed=11)


def test_ragged_batch_routing_and_graph_replay_lag():
    roles = [[T, F], [A, T], [T, T], [T, F], [A, F], [F, F], [T, F]]
    w = tiny_custom(n_layers=7, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=9, audio_lens=(400, 75, 1000), chunk=25,
                    budget=0.2, n_steps=12, roles=roles, region=50, jump_every=4)
    _run(w, delta=3, seed=4, graph_from=2)


@pytest.mark.parametrize("dependency", [1, 2])
def test_chained_and_serial_layers_lag(dependency):
    roles = [[A, T, T, F], [T, F, T, F], [A, T, F, T]]
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640, 300), chunk=25, budget=0.2,
                    n_steps=8, roles=roles, region=32, jump_every=3)
    _run(w, delta=2, seed=8, graph_from=1, dependency=dependency)


def test_global_scope_lag():
    roles = [[T, F], [A, T], [A, A], [T, T], [A, F]]
    w = tiny_custom(n_layers=5, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=9, audio_lens=(500, 130), chunk=25,
                    budget=0.25, n_steps=8, roles=roles, region=25, jump_every=3)
    _run(w, delta=3, seed=5, graph_from=3, scope=1)


def test_pool_size_and_release_counts_lag():
    """The dynamic pool is 2k(delta+1) slots and is never short; with a jumping focus segments are fetched and released."""
    roles = [[A, T, T, F], [A, T, F, T]]
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=8, audio_lens=(2000,), chunk=25, budget=0.1,
                    n_steps=16, roles=roles, region=25, jump_every=2)
    ls = _run(w, delta=3, seed=2, graph_from=4)
    st = ls.o.stats(0) if ls.o._h else None   # the counters were compared with the oracle's in check_stats


def test_config1_shape_with_paper_segments_graph_replay():
    """3B Voxtral-shaped stack with the paper's segment length (25 tokens: 120 segments, 119 chunks), 12 replayed steps."""
    w = config1(n_steps=12)
    w.chunk = 25
    _run(w, delta=3, graph_from=1, check_slots=False)


def test_residency_rejects_unknown_value():
    from workloads import config0
    w = config0()
    with pytest.raises(wnw.WnwError):
        wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, 1024, w.text_capacity, w.chunk, w.budget,
                       w.roles, topk=w.topk, residency=5)
