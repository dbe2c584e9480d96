"""Replayed steps issued back to back, with no host synchronisation between them: the recall of a step then runs
outside the captured graph and overlaps the next step, whose tidal CTAs wait on per-layer epoch words.  The result must
be bit-identical to the same steps drained one by one (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_TIDAL, Synth, config1, config4

pytestmark = pytest.mark.gpu


def _run(w, drained, n_steps, dependency=0, score_scope=0, eager_steps=(), residency=0):
    dev = torch.device("cuda:0")
    syn = Synth(w, seed=3, device="cuda:0")
    h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(w.audio_lens), w.text_capacity,
                       w.chunk, w.budget, w.roles, topk=w.topk, score_scope=score_scope, residency=residency, evict_lag=2)
    try:
        wnw.wnw_set_layer_dependency(h, dependency)
        for b in range(w.batch):
            for l in range(w.n_layers):
                p = syn.prefill(b, l)
                wnw.wnw_place_prefill(h, b, l, p["k"], p["v"], p["audio_begin"], p["audio_end"], p["q_last"])
                torch.cuda.synchronize()
        dec = {(b, l): syn.decode(b, l) for b in range(w.batch) for l in range(w.n_layers)}
        q = torch.stack([torch.stack([torch.stack([dec[(b, l)]["q"][t] for b in range(w.batch)]) for l in range(w.n_layers)])
                         for t in range(n_steps)])
        kn = torch.stack([torch.stack([torch.stack([dec[(b, l)]["k_new"][t] for b in range(w.batch)]) for l in range(w.n_layers)])
                          for t in range(n_steps)])
        vn = torch.stack([torch.stack([torch.stack([dec[(b, l)]["v_new"][t] for b in range(w.batch)]) for l in range(w.n_layers)])
                          for t in range(n_steps)])
        sq, skn, svn = torch.empty_like(q[0]), torch.empty_like(kn[0]), torch.empty_like(vn[0])
        out = torch.zeros_like(q[0])
        st = torch.cuda.Stream(device=dev)
        torch.cuda.synchronize()
        act = list(range(w.batch))
        wnw.wnw_graph_begin(h, act, st)
        wnw.wnw_step_begin(h, act)
        for l in range(w.n_layers):
            wnw.wnw_decode_layer(h, l, sq[l], skn[l], svn[l], out[l], stream=st)
        wnw.wnw_step_end(h, stream=st)
        wnw.wnw_graph_end(h, st)
        outs = []
        with torch.cuda.stream(st):
            for t in range(n_steps):
                sq.copy_(q[t]); skn.copy_(kn[t]); svn.copy_(vn[t])
                if t in eager_steps:       # an eager step between replays, on the same stream, still without host sync
                    wnw.wnw_step_begin(h, act)
                    for l in range(w.n_layers):
                        wnw.wnw_decode_layer(h, l, sq[l], skn[l], svn[l], out[l], stream=st)
                    wnw.wnw_step_end(h, stream=st)
                else:
                    wnw.wnw_graph_launch(h, st)
                outs.append(out.clone())
                if drained:
                    wnw.wnw_sync(h)
        torch.cuda.synchronize()
        wnw.wnw_sync(h)
        tabs = [wnw.wnw_get_residency(h, b, l) for b in range(w.batch) for l in range(w.n_layers)
                if (w.roles[l] == ROLE_TIDAL).any()]
        return outs, tabs, wnw.wnw_get_stats(h), wnw.wnw_get_launch_counts(h)
    finally:
        wnw.wnw_destroy(h)


def _same(a, b):
    for t, (x, y) in enumerate(zip(a[0], b[0])):
        if not torch.equal(x, y):
            d = (x.float() - y.float()).abs()
            where = [(l, b, h) for l in range(x.shape[0]) for b in range(x.shape[1]) for h in range(x.shape[2])
                     if d[l, b, h].max() > 0]
            raise AssertionError(f"outputs differ at step {t}: max abs {d.max().item():.4g}, (layer, seq, q head) {where[:12]}")
    for (t1, s1), (t2, s2) in zip(a[1], b[1]):
        assert np.array_equal(t1, t2) and np.array_equal(s1, s2)
    assert a[2] == b[2]


@pytest.mark.parametrize("budget,chunk,batch", [(0.2, 64, 1), (0.4, 64, 2), (0.4, 256, 4)])
def test_undrained_replays_match_drained(budget, chunk, batch):
    """Jumping focus (misses in every layer at once every fourth step): long recalls overlap the following steps."""
    w = config4(budget=budget, chunk=chunk, batch=batch, n_steps=12)
    w.n_layers = 8; w.roles = w.roles[:8]
    a = _run(w, True, 12)
    b = _run(w, False, 12)
    _same(a, b)
    assert a[2]["misses"] > 0 and a[2]["recall_bytes"] > 0
    attn, sel, rec, end = b[3]
    assert attn == 12 * w.n_layers and rec == 12 and end == 0     # one recall launch per replayed step, no step-end kernel


def test_undrained_replays_match_drained_config1_shape_and_scopes():
    w = config1(n_steps=10)
    w.n_layers = 10; w.roles = w.roles[:10]
    for scope in (0, 1):
        _same(_run(w, True, 10, score_scope=scope), _run(w, False, 10, score_scope=scope))


@pytest.mark.parametrize("dependency", [1, 2])
def test_undrained_replays_match_drained_chained_and_serial(dependency):
    w = config4(budget=0.2, chunk=64, batch=2, n_steps=8)
    w.n_layers = 6; w.roles = w.roles[:6]
    _same(_run(w, True, 8, dependency=dependency), _run(w, False, 8, dependency=dependency))


@pytest.mark.parametrize("residency", [0, 1])
def test_undrained_mix_of_eager_steps_and_replays(residency):
    """Eager steps in between replays on the same stream, nothing drained: the eager step waits for the pending
    out-of-graph recall, the next replay for the eager step's side streams."""
    w = config4(budget=0.2, chunk=25 if residency else 64, batch=2, n_steps=12)
    w.n_layers = 6; w.roles = w.roles[:6]
    a = _run(w, True, 12, eager_steps=(3, 4, 8), residency=residency)
    b = _run(w, False, 12, eager_steps=(3, 4, 8), residency=residency)
    _same(a, b)
    c = _run(w, False, 12, residency=residency)          # and the mix gives what pure replay gives
    for t, (x, y) in enumerate(zip(a[0], c[0])):
        assert torch.equal(x, y), (f"eager/replay mix differs from pure replay at step {t}: max abs "
                                   f"{(x.float() - y.float()).abs().max().item():.4g}, layers "
                                   f"{[l for l in range(w.n_layers) if not torch.equal(x[l], y[l])]}")


@pytest.mark.parametrize("dependency,residency", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_undrained_replays_large_launches(dependency, residency):
    """Launches too large for the out-of-graph recall (recall stays inside the captured step); chained layers run the
    persistent schedule.  Eager steps mixed in."""
    w = config4(budget=0.1, chunk=25 if residency else 64, batch=12, n_steps=8)
    w.n_layers = 4; w.roles = w.roles[:4]
    a = _run(w, True, 8, dependency=dependency, residency=residency, eager_steps=(2, 5))
    b = _run(w, False, 8, dependency=dependency, residency=residency, eager_steps=(2, 5))
    _same(a, b)
    assert b[3][2] > 8      # recall launches per layer, not one per step


@pytest.mark.parametrize("budget,chunk,batch,residency", [(0.2, 64, 1, 0), (0.4, 64, 2, 0), (0.2, 25, 2, 1), (0.4, 256, 3, 0)])
def test_undrained_batched_replays_match_drained(budget, chunk, batch, residency):
    """All layers issued together (BATCHED): the step's selection runs beside its tidal attention and the recall of the
    previous step beside both; nothing drained between 16 replays, focus jumping every fourth step (long recalls)."""
    w = config4(budget=budget, chunk=chunk, batch=batch, n_steps=16)
    w.n_layers = 8; w.roles = w.roles[:8]
    a = _run(w, True, 16, dependency=3, residency=residency)
    b = _run(w, False, 16, dependency=3, residency=residency)
    _same(a, b)
    assert a[2]["misses"] > 0 and a[2]["recall_bytes"] > 0
    attn, sel, rec, end = b[3]
    assert attn == 3 * 16 and rec == 16 and end == 16     # three attention launches, one recall, one step-end kernel per replay
    c = _run(w, False, 16, dependency=0, residency=residency)      # and the per-layer launches give the same tables
    for (t1, s1), (t2, s2) in zip(a[1], c[1]):
        assert np.array_equal(t1, t2) and np.array_equal(s1, s2)
    assert a[2] == c[2]


def test_undrained_batched_mix_of_eager_steps_and_replays():
    w = config1(n_steps=14)
    w.n_layers = 10; w.roles = w.roles[:10]
    for scope in (0, 1):
        a = _run(w, True, 14, dependency=3, score_scope=scope, eager_steps=(3, 4, 9))
        b = _run(w, False, 14, dependency=3, score_scope=scope, eager_steps=(3, 4, 9))
        _same(a, b)


def test_undrained_batched_config1_full_stack():
    """Config 1 at full size (30 layers), 64 replays with nothing drained in between, all layers issued together: the
    outputs, tables and counters of the drained run."""
    w = config1(n_steps=64)
    a = _run(w, True, 64, dependency=3)
    b = _run(w, False, 64, dependency=3)
    _same(a, b)
    assert a[2]["misses"] > 0
