"""Sequences joining and leaving between steps: every step serves its own active set, a finished sequence's slot is
re-placed with a fresh prefill while the others keep decoding, and captured steps are re-captured when the set changes.
Everything in lock-step with the oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, tiny_custom
from workloads.synth import bf16_bits

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _replace(ls, b):
    """Places sequence b's prefill again (a new request taking over the slot): state, tables and counters start over."""
    w = ls.w
    for l in range(w.n_layers):
        p = ls.syn.prefill(b, l)
        k, v, ql = (p[n].to(ls.dev) for n in ("k", "v", "q_last"))
        wnw.wnw_place_prefill(ls.h, b, l, k, v, p["audio_begin"], p["audio_end"], ql)
        ls.o.place_prefill(b, l, bf16_bits(p["k"]), bf16_bits(p["v"]), p["audio_begin"], p["audio_end"], bf16_bits(p["q_last"]))
    wnw.wnw_sync(ls.h)
    ls._steps[b] = 0
    for l in range(w.n_layers):
        if (w.roles[l] == T).any():
            g_tab, g_stamp = wnw.wnw_get_residency(ls.h, b, l)
            o_tab, o_stamp = ls.o.residency(b, l)
            assert g_tab.tolist() == o_tab.tolist() and g_stamp.tolist() == o_stamp.tolist()
    assert wnw.wnw_get_seq_dims(ls.h, b) == ls.o.dims(b)


@pytest.mark.parametrize("residency", [0, 1])
def test_sequences_join_leave_and_slots_are_reused(residency):
    from parity_harness import Lockstep
    roles = [[A, T, T, F], [T, F, T, F], [A, T, F, T]]
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(400, 170, 640, 90), chunk=25,
                    budget=0.2, n_steps=14, roles=roles, region=25, jump_every=3)
    ls = Lockstep(w, seed=21, residency=residency, evict_lag=2)
    try:
        ls.prefill()
        schedule = [[0, 1, 2, 3], [0, 1, 2, 3], [0, 2, 3], [0, 2], [2], [2, 1], [1, 2, 3], [3, 1, 2, 0], [0], [0, 1, 2, 3]]
        for t, act in enumerate(schedule):
            if t == 5:
                _replace(ls, 1)          # sequence 1 left after step 1; a new request takes its slot
            if t == 8:
                _replace(ls, 3)
            ls.decode_step(t, active=act, check_slots=True)
        # per-sequence step counts: what each slot decoded since its last placement
        assert ls._steps == {0: 7, 1: 4, 2: 9, 3: 1}
        for b in range(4):
            T_a, T_t, C, S = wnw.wnw_get_seq_dims(ls.h, b)
            assert T_t == w.n_text + ls._steps[b]
    finally:
        ls.close()


def test_graph_is_recaptured_when_the_active_set_changes():
    from parity_harness import Lockstep
    roles = [[A, T], [T, F]]
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=4, audio_lens=(300, 200, 500), chunk=16,
                    budget=0.25, n_steps=10, roles=roles)
    ls = Lockstep(w, seed=5)
    try:
        ls.prefill()
        ls.decode_step(0, active=[0, 1, 2], graph=True, check_slots=True)
        ls.decode_step(1, active=[0, 1, 2], graph=True, check_slots=True)
        ls.decode_step(2, active=[0, 2], check_slots=True)            # eager step of another set: the work lists change
        with pytest.raises(wnw.WnwError):                             # the captured step is stale now: refused, not replayed
            wnw.wnw_graph_launch(ls.h, ls._gstream)
        for t, act in enumerate([[0, 2], [2, 1], [2, 1], [1], [1]], start=3):
            if t in (3, 4, 6):
                ls._graph = None                                      # capture again for the new set
            ls.decode_step(t, active=act, graph=True, check_slots=True)
    finally:
        ls.close()
