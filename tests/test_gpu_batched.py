"""BATCHED layers: inside a captured step the attention of all layers runs as one launch that carries the CTAs of every
layer (three with all head roles: the anchor heads, behind which the step's selection is forked, the fixed heads, the
tidal heads).  Parity against the oracle in the
replayed configuration, against the per-layer launches, and the fallbacks.  Needs a B200."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, config1, config2, tiny_custom

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _tiny():
    return tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640, 300), chunk=32, budget=0.2,
                       n_steps=12, roles=[[A, T, T, F], [T, F, T, F], [A, T, F, T]], region=32, jump_every=3)


def test_batched_replay_matches_oracle_and_counts_three_attention_launches_per_step():
    from parity_harness import Lockstep
    ls = Lockstep(_tiny(), seed=8)
    try:
        wnw.wnw_set_layer_dependency(ls.h, wnw.WNW_LAYERS_BATCHED)
        ls.prefill()
        ls.decode_step(0, check_slots=True)                       # eager: per-layer launches (the mode's fallback)
        c0 = wnw.wnw_get_launch_counts(ls.h)
        for t in range(1, 7):
            ls.decode_step(t, graph=True, check_slots=True)       # replays: anchor heads, fixed heads, tidal heads
        c1 = wnw.wnw_get_launch_counts(ls.h)
        assert c1[0] - c0[0] == 3 * 6
        ls.decode_step(7, check_slots=True)
        for t in range(8, 12):
            ls.decode_step(t, graph=True, check_slots=True)
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


@pytest.mark.parametrize("cfg,steps", [(config1, 24), (config2, 8)])
def test_batched_full_size_graph_replay(cfg, steps):
    """Configs 1 and 2 at full size, every step replayed with all layers in one launch; the oracle follows every step."""
    from parity_harness import Lockstep
    w = cfg(n_steps=steps)
    ls = Lockstep(w, seed=0, gen_device="cuda:0")
    try:
        wnw.wnw_set_layer_dependency(ls.h, wnw.WNW_LAYERS_BATCHED)
        ls.prefill(check_slots=False)
        for t in range(steps):
            ls.decode_step(t, graph=True, check_slots=(t == steps - 1))
        ls.check_stats()
        c = wnw.wnw_get_launch_counts(ls.h)
        assert c[0] == 3 * steps
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_batched_with_token_base_and_global_scope():
    from parity_harness import Lockstep
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=9, audio_lens=(640, 300, 77), chunk=25, budget=0.3,
                    n_steps=8, roles=[[A, T, F, T], [T, F, T, F], [A, T, T, T]], region=25, jump_every=3, topk=2)
    w.n_prefill_queries = 2
    ret = np.array([[1.0, 0.3, 0.45, 0.0], [0.5, 0.2, 0.08, 0.33], [1.0, 0.41, 0.25, 0.5]], np.float32)
    ls = Lockstep(w, seed=12, score_scope=1, residency=2, evict_lag=1, token_retention=ret, token_seg=25)
    try:
        wnw.wnw_set_layer_dependency(ls.h, wnw.WNW_LAYERS_BATCHED)
        ls.prefill()
        for t in range(8):
            ls.decode_step(t, graph=(t > 0), check_slots=True)
        ls.check_stats()
        assert ls.max_out_err <= 2e-2
    finally:
        ls.close()


def test_batched_agrees_with_per_layer_launches_in_full_cache_mode():
    """FULL mode has no oracle-side tables to compare: the batched replay must give the outputs of the per-layer replay
    (same work, different cut: equal up to the rounding order of the split merge)."""
    from workloads import Synth
    w = tiny_custom(n_layers=4, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=6, audio_lens=(900, 333), chunk=32, budget=0.2,
                    n_steps=5)
    outs = {}
    for dep in (wnw.WNW_LAYERS_INDEPENDENT, wnw.WNW_LAYERS_BATCHED):
        syn = Synth(w, seed=5, device="cuda:0")
        h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(w.audio_lens), w.text_capacity, w.chunk,
                           w.budget, w.roles, topk=w.topk, mode=wnw.WNW_MODE_FULL)
        try:
            wnw.wnw_set_layer_dependency(h, dep)
            for b in range(w.batch):
                for l in range(w.n_layers):
                    p = syn.prefill(b, l)
                    wnw.wnw_place_prefill(h, b, l, p["k"], p["v"], p["audio_begin"], p["audio_end"], p["q_last"])
                    torch.cuda.synchronize()
            dec = {(b, l): syn.decode(b, l) for b in range(w.batch) for l in range(w.n_layers)}
            q = torch.zeros(w.n_layers, w.batch, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
            kn = torch.zeros(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
            vn = torch.zeros_like(kn)
            out = torch.zeros_like(q)
            res = []
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for t in range(w.n_steps):
                    for l in range(w.n_layers):
                        for b in range(w.batch):
                            q[l, b], kn[l, b], vn[l, b] = dec[(b, l)]["q"][t], dec[(b, l)]["k_new"][t], dec[(b, l)]["v_new"][t]
                    if t == 0:
                        st.synchronize()
                        wnw.wnw_graph_begin(h, list(range(w.batch)), stream=st)
                        wnw.wnw_step_begin(h, list(range(w.batch)))
                        for l in range(w.n_layers):
                            wnw.wnw_decode_layer_full(h, l, q[l], kn[l], vn[l], out[l], stream=st)
                        wnw.wnw_step_end(h, stream=st)
                        wnw.wnw_graph_end(h, stream=st)
                    wnw.wnw_graph_launch(h, stream=st)
                    st.synchronize()
                    res.append(out.float().cpu().numpy().copy())
            outs[dep] = res
            if dep == wnw.WNW_LAYERS_BATCHED:
                assert wnw.wnw_get_launch_counts(h)[0] == w.n_steps
        finally:
            wnw.wnw_destroy(h)
    for a, b in zip(outs[wnw.WNW_LAYERS_INDEPENDENT], outs[wnw.WNW_LAYERS_BATCHED]):
        assert np.abs(a - b).max() <= 2e-2
        assert np.abs(a).max() > 0
