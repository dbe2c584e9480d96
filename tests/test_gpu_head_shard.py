"""Head-sharded serving on the GPU library: shards of the KV heads as separate caches, the chunk-score exchange between
them, against ONE oracle that holds every head.  This box has one GPU, so the shards run one after the other on it and
the all-reduce is a sum of their exported buffers (no kernel waits on another); with one process per GPU the same calls
run with torch.distributed.all_reduce in between (paper_2608_22704_b200.sharded.sharded_step).  Needs a B200."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from helpers import bf16_bits_to_f64, dequantised_tidal_bits, make_oracle
from oracle import wnw_oracle as wo
from paper_2608_22704_b200.sharded import create_shard_cache, shard_plan, sharded_step
from parity_harness import OUT_TOL, assert_scores_close, chunk_lens
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, tiny_custom
from workloads.synth import bf16_bits

pytestmark = pytest.mark.gpu
A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED


def _run(roles, world, n_steps=6, seed=13, kv_fp8=False):
    """kv_fp8: the shards keep their tidal tier as e4m3 (head_dim 128); the oracle gets the values the bytes decode to."""
    w = tiny_custom(n_layers=len(roles), n_q_heads=8, n_kv_heads=4, head_dim=128 if kv_fp8 else 64, n_text=6, audio_lens=(200, 90),
                    chunk=16, budget=0.3, n_steps=n_steps, roles=roles, region=16)
    dev = torch.device("cuda:0")
    syn = Synth(w, seed=seed)
    o = make_oracle(w)
    plan = shard_plan(w.roles, w.n_q_heads, world)
    caches = [create_shard_cache(sh, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(w.audio_lens), w.text_capacity, w.chunk,
                                 w.budget, topk=w.topk,
                                 tidal_kv_format=wnw.WNW_TIDAL_KV_FP8_E4M3 if kv_fp8 else wnw.WNW_TIDAL_KV_BF16) for sh in plan]
    C_max = -(-max(w.audio_lens) // w.chunk)
    try:
        # ---- placement, with the exchange of the tidal heads' prefill sums per (sequence, layer)
        for b in range(w.batch):
            for l in range(w.n_layers):
                p = syn.prefill(b, l)
                kb, vb = bf16_bits(p["k"]), bf16_bits(p["v"])
                if kv_fp8:
                    kb, vb = dequantised_tidal_bits(kb, vb, w.roles[l], p["audio_begin"], p["audio_end"], w.chunk)
                o.place_prefill(b, l, kb, vb, p["audio_begin"], p["audio_end"], bf16_bits(p["q_last"]))
                sums = []
                for sh, h in zip(plan, caches):
                    wnw.wnw_place_prefill(h, b, l, p["k"][:, sh.kv_heads].contiguous().to(dev), p["v"][:, sh.kv_heads].contiguous().to(dev),
                                          p["audio_begin"], p["audio_end"], p["q_last"][sh.q_heads].contiguous().to(dev))
                    s_ = torch.zeros(C_max, dtype=torch.float32, device=dev)
                    wnw.wnw_export_prefill_tidal(h, b, l, s_)
                    sums.append(s_)
                total = torch.stack(sums).sum(0)                   # what the all-reduce leaves on every rank
                for h in caches:
                    wnw.wnw_import_prefill_tidal(h, b, l, total)
                torch.cuda.synchronize()
                T_a, _, C, S = o.dims(b)
                if (w.roles[l] == T).any():
                    want = wo.topk(total.cpu().numpy()[:C], chunk_lens(T_a, w.chunk), S).tolist()
                    for sh, h in zip(plan, caches):
                        if (sh.roles[l] == T).any():
                            tab, stamp = wnw.wnw_get_residency(h, b, l)
                            assert tab.tolist() == want and tab.tolist() == o.residency(b, l)[0].tolist()
                            assert stamp.tolist() == [-1 - r for r in range(S)]
        dec = {(b, l): syn.decode(b, l) for b in range(w.batch) for l in range(w.n_layers)}
        act = list(range(w.batch))
        max_err = 0.0
        for t in range(n_steps):
            o.step_begin(act)
            ref = [o.decode_layer(l, np.stack([bf16_bits(dec[(b, l)]["q"][t]) for b in act]),
                                  np.stack([bf16_bits(dec[(b, l)]["k_new"][t]) for b in act]),
                                  np.stack([bf16_bits(dec[(b, l)]["v_new"][t]) for b in act])) for l in range(w.n_layers)]
            outs, exported = [], []
            for sh, h in zip(plan, caches):                        # every shard up to its export
                q = [torch.stack([dec[(b, l)]["q"][t][sh.q_heads] for b in act]).to(dev) for l in range(w.n_layers)]
                kn = [torch.stack([dec[(b, l)]["k_new"][t][sh.kv_heads] for b in act]).to(dev) for l in range(w.n_layers)]
                vn = [torch.stack([dec[(b, l)]["v_new"][t][sh.kv_heads] for b in act]).to(dev) for l in range(w.n_layers)]
                out = [torch.full_like(x, float("nan")) for x in q]
                wnw.wnw_step_begin(h, act)
                for l in range(w.n_layers):
                    wnw.wnw_decode_layer(h, l, q[l], kn[l], vn[l], out[l])
                sc = torch.zeros((len(act), w.n_layers, C_max), dtype=torch.float32, device=dev)
                wnw.wnw_export_scores(h, sc)
                outs.append(out); exported.append(sc)
            total = torch.stack(exported).sum(0)                    # the all-reduce
            for h in caches:
                wnw.wnw_import_scores(h, total)
                wnw.wnw_step_end(h)
                wnw.wnw_sync(h)
            o.step_end()
            tot = total.cpu().numpy()
            for r, (sh, h) in enumerate(zip(plan, caches)):
                for l in range(w.n_layers):
                    got = bf16_bits_to_f64(bf16_bits(outs[r][l].cpu()))
                    err = float(np.abs(got - ref[l][:, sh.q_heads]).max())
                    max_err = max(max_err, err)
                    assert err <= OUT_TOL, (t, r, l, err)
                    for i, b in enumerate(act):
                        T_a, _, C, S = o.dims(b)
                        if (w.roles[l] == A).any():
                            assert_scores_close(tot[i, l, :C], o.chunk_scores(b, l), f"summed scores step {t} b{b} l{l}")
                        if (sh.roles[l] == T).any():
                            src = o.score_source(l)
                            want = wo.topk(tot[i, src, :C], chunk_lens(T_a, w.chunk), min(w.topk, S)).tolist()
                            assert wnw.wnw_get_selected(h, b, l).tolist() == want == o.selected(b, l).tolist(), (t, r, l, b)
                            tab, stamp = wnw.wnw_get_residency(h, b, l)
                            otab, ostamp = o.residency(b, l)
                            assert tab.tolist() == otab.tolist() and stamp.tolist() == ostamp.tolist(), (t, r, l, b)
        return max_err
    finally:
        for h in caches:
            wnw.wnw_destroy(h)
        o.close()


@pytest.mark.parametrize("world", [2, 4])
def test_head_shards_match_one_oracle(world):
    """Anchor heads of a layer on one shard (the others contribute zero rows), layers without any anchor routed by the
    model-wide flags, tidal heads of one layer spread over the shards (one table, ranked by the sum over all of them)."""
    assert _run([[A, T, T, F], [T, F, T, T], [F, T, A, T]], world) > 0


def test_head_shards_with_an_e4m3_tidal_tier():
    """The shards' slots are refilled from e4m3 mirrors after the exchange of the prefill sums."""
    assert _run([[A, T, T, F], [T, F, T, T], [F, T, A, T]], 2, kv_fp8=True) > 0


def test_head_shards_with_a_layers_anchor_heads_split_over_shards():
    assert _run([[A, T, A, T], [T, F, T, T], [F, A, T, A]], 2) > 0


def test_one_shard_with_deferred_selection_is_the_ordinary_cache():
    """world = 1 through sharded_step (the all-reduce is the identity): deferring the selection to the end of the step
    changes nothing (a selection is used from the next step on either way)."""
    w = tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(200,), chunk=16, budget=0.3, n_steps=5,
                    roles=[[A, T, T, F], [T, F, T, T], [F, T, A, T]], region=16)
    dev = torch.device("cuda:0")
    syn = Synth(w, seed=3)
    o = make_oracle(w)
    sh = shard_plan(w.roles, w.n_q_heads, 1)[0]
    h = create_shard_cache(sh, w.n_q_heads, w.n_kv_heads, w.head_dim, 1, 200, w.text_capacity, w.chunk, w.budget, topk=w.topk)
    try:
        for l in range(w.n_layers):
            p = syn.prefill(0, l)
            wnw.wnw_place_prefill(h, 0, l, p["k"].to(dev), p["v"].to(dev), p["audio_begin"], p["audio_end"], p["q_last"].to(dev))
            o.place_prefill(0, l, bf16_bits(p["k"]), bf16_bits(p["v"]), p["audio_begin"], p["audio_end"], bf16_bits(p["q_last"]))
        dec = [syn.decode(0, l) for l in range(w.n_layers)]
        scores = torch.zeros((1, w.n_layers, -(-200 // 16)), dtype=torch.float32, device=dev)
        for t in range(w.n_steps):
            q = [dec[l]["q"][t][None].to(dev) for l in range(w.n_layers)]
            kn = [dec[l]["k_new"][t][None].to(dev) for l in range(w.n_layers)]
            vn = [dec[l]["v_new"][t][None].to(dev) for l in range(w.n_layers)]
            out = [torch.empty_like(x) for x in q]
            sharded_step(h, [0], q, kn, vn, out, scores, all_reduce=lambda x: x)
            wnw.wnw_sync(h)
            o.step_begin([0])
            for l in range(w.n_layers):
                ref = o.decode_layer(l, bf16_bits(q[l].cpu()), bf16_bits(kn[l].cpu()), bf16_bits(vn[l].cpu()))
                assert np.abs(bf16_bits_to_f64(bf16_bits(out[l].cpu())) - ref).max() <= OUT_TOL
            o.step_end()
            for l in range(w.n_layers):
                if (w.roles[l] == T).any():
                    assert wnw.wnw_get_selected(h, 0, l).tolist() == o.selected(0, l).tolist()
                    assert wnw.wnw_get_residency(h, 0, l)[0].tolist() == o.residency(0, l)[0].tolist()
    finally:
        wnw.wnw_destroy(h)
        o.close()
