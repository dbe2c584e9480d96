"""GPU parity for the global score scope (Eq. 2 as printed): one accumulator over every anchor (layer, q-head) pair of
the step, one selection shared by all tidal layers, made after the last layer of the step (needs a B200)."""
import numpy as np
import pytest

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, config0, config1, tiny_custom

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _run(w, n_steps=None, seed=0, graph_from=None, check_slots=True, recall_mode=0):
    from parity_harness import Lockstep
    ls = Lockstep(w, seed=seed, score_scope=wnw.WNW_SCOPE_GLOBAL, recall_mode=recall_mode)
    try:
        ls.prefill(check_slots=check_slots)
        for t in range(w.n_steps if n_steps is None else n_steps):
            ls.decode_step(t, graph=graph_from is not None and t >= graph_from, check_slots=check_slots)
        ls.check_stats()
        # every tidal layer of a sequence carries the same selection
        for b in range(w.batch):
            sels = [wnw.wnw_get_selected(ls.h, b, l).tolist() for l in range(w.n_layers) if (w.roles[l] == T).any()]
            assert all(s == sels[0] for s in sels)
        return ls
    finally:
        ls.close()


@pytest.mark.parametrize("graph_from", [None, 1])
def test_global_scope_mixed_layers(graph_from):
    """Anchor-only, tidal-only and mixed layers; the last layer has no anchor head, so its tail only sums and selects."""
    roles = [[T, F], [A, T], [A, A], [T, T], [A, F], [F, F], [T, F]]
    w = tiny_custom(n_layers=7, n_q_heads=8, n_kv_heads=2, head_dim=64, n_text=9, audio_lens=(160, 75, 512), chunk=16,
                    budget=0.25, n_steps=8, roles=roles)
    _run(w, seed=4, graph_from=graph_from)


def test_global_scope_last_layer_has_anchor_and_paper_chunk():
    roles = [[A, T, T, F], [T, F, T, F], [A, T, F, T]]
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640, 300), chunk=50, budget=0.2,
                    n_steps=10, roles=roles, region=32, jump_every=3)
    _run(w, seed=8, graph_from=2)


def test_global_scope_more_tidal_layers_than_select_warps():
    """Twelve tidal layers updated by one tail: more than the warps of the selection CTA and more than the by-value list."""
    roles = [[A, T]] * 12
    w = tiny_custom(n_layers=12, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(300, 41), chunk=16, budget=0.2,
                    n_steps=6, roles=roles, region=16, jump_every=2)
    _run(w, seed=3, graph_from=3)


def test_global_scope_single_layer_equals_per_layer():
    """With one layer the two scopes coincide: same selections and tables step by step."""
    from parity_harness import Lockstep
    w = config0()
    a, b = Lockstep(w, seed=0, score_scope=0), Lockstep(w, seed=0, score_scope=1)
    try:
        a.prefill(); b.prefill()
        for t in range(8):
            a.decode_step(t); b.decode_step(t)
            assert wnw.wnw_get_selected(a.h, 0, 0).tolist() == wnw.wnw_get_selected(b.h, 0, 0).tolist()
            ta, tb = wnw.wnw_get_residency(a.h, 0, 0), wnw.wnw_get_residency(b.h, 0, 0)
            assert np.array_equal(ta[0], tb[0]) and np.array_equal(ta[1], tb[1])
    finally:
        a.close(); b.close()


def test_global_scope_config1_graph_steps():
    """3B Voxtral-shaped stack under graph replay, global scope: 30 tidal layers updated by the last layer's tail."""
    _run(config1(), n_steps=6, graph_from=1, check_slots=False)


def test_global_scope_rejects_unknown_value():
    w = config0()
    with pytest.raises(wnw.WnwError):
        wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, 1024, w.text_capacity, w.chunk, w.budget,
                       w.roles, topk=w.topk, score_scope=7)
