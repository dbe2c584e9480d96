"""Head-sharded serving on CPU: two gloo ranks, each an oracle over its own KV heads, one all-reduce of the chunk scores
per step.  The shards' outputs, the summed scores, the selections and the residency tables must be those of one oracle
holding every head: bit for bit where every layer's anchor heads sit on one rank (the other rank adds zeros), to rounding
of the last bit of a double sum where they are split (then selections and tables are still compared exactly)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
A, T, F = 0, 1, 2


def _workload(split_anchors):
    from workloads import tiny_custom
    roles = [[A, T, T, F], [T, F, T, T], [F, T, A, T]] if not split_anchors else [[A, T, A, T], [T, F, T, T], [F, A, T, A]]
    return tiny_custom(n_layers=3, n_q_heads=8, n_kv_heads=4, head_dim=64, n_text=6, audio_lens=(200, 90), chunk=16, budget=0.3,
                       n_steps=6, roles=roles, region=16)


def _run_reference(w, seed):
    """One oracle with every head: per step outputs, scores, selections, tables."""
    from helpers import make_oracle, place_all
    from workloads import Synth
    from workloads.synth import bf16_bits
    syn = Synth(w, seed=seed)
    o = make_oracle(w)
    place_all(o, syn)
    dec = {(b, l): syn.decode(b, l) for b in range(w.batch) for l in range(w.n_layers)}
    trace = []
    for t in range(w.n_steps):
        o.step_begin(list(range(w.batch)))
        outs = []
        for l in range(w.n_layers):
            q = np.stack([bf16_bits(dec[(b, l)]["q"][t]) for b in range(w.batch)])
            kn = np.stack([bf16_bits(dec[(b, l)]["k_new"][t]) for b in range(w.batch)])
            vn = np.stack([bf16_bits(dec[(b, l)]["v_new"][t]) for b in range(w.batch)])
            outs.append(o.decode_layer(l, q, kn, vn))
        scores = {(b, l): o.chunk_scores(b, l).copy() for b in range(w.batch) for l in range(w.n_layers)}
        o.step_end()
        trace.append({"out": outs, "scores": scores,
                      "sel": {(b, l): o.selected(b, l).tolist() for b in range(w.batch) for l in range(w.n_layers)},
                      "tab": {(b, l): [x.tolist() for x in o.residency(b, l)] for b in range(w.batch) for l in range(w.n_layers)}})
    o.close()
    return trace


def _worker(rank, world, port, split_anchors, seed, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    for p in (ROOT, os.path.join(ROOT, "tests")):
        if p not in sys.path:
            sys.path.insert(0, p)
    from oracle.wnw_oracle import Oracle
    from paper_2608_22704_b200.sharded import shard_plan
    from workloads import Synth
    from workloads.synth import bf16_bits
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = _workload(split_anchors)
        sh = shard_plan(w.roles, w.n_q_heads, world)[rank]
        g = w.n_q_heads // w.n_kv_heads
        o = Oracle(w.n_layers, len(sh.kv_heads) * g, len(sh.kv_heads), w.head_dim, w.batch, max(w.audio_lens), w.text_capacity, w.chunk,
                   w.topk, w.budget, sh.roles, global_anchor_layers=sh.global_anchor_layers)
        syn = Synth(w, seed=seed)
        for b in range(w.batch):
            for l in range(w.n_layers):
                p = syn.prefill(b, l)
                o.place_prefill(b, l, bf16_bits(p["k"])[:, sh.kv_heads], bf16_bits(p["v"])[:, sh.kv_heads], p["audio_begin"], p["audio_end"],
                                bf16_bits(p["q_last"])[sh.q_heads])
        # a layer's tidal table starts from the prefill score summed over ALL its tidal heads: the same exchange at placement
        from oracle import wnw_oracle as wo
        for b in range(w.batch):
            T_a, _, C, S = o.dims(b)
            lens = np.array([min(w.chunk, T_a - c * w.chunk) for c in range(C)], np.int32)
            for l in range(w.n_layers):
                buf = torch.zeros(C, dtype=torch.float64)
                for j in range(len(sh.kv_heads)):
                    if sh.roles[l, j] == T:
                        buf += torch.from_numpy(o.prefill_scores(b, l, j))
                dist.all_reduce(buf)
                if (sh.roles[l] == T).any():
                    top = wo.topk(buf.numpy().astype(np.float32), lens, S)
                    tab = np.full(S, -1, np.int32); stamp = np.zeros(S, np.int64)
                    tab[:len(top)] = top; stamp[:len(top)] = -1 - np.arange(len(top))
                    o.set_residency(b, l, tab, stamp)
        dec = {(b, l): syn.decode(b, l) for b in range(w.batch) for l in range(w.n_layers)}
        trace = []
        for t in range(w.n_steps):
            o.step_begin(list(range(w.batch)))
            outs = []
            for l in range(w.n_layers):
                q = np.stack([bf16_bits(dec[(b, l)]["q"][t])[sh.q_heads] for b in range(w.batch)])
                kn = np.stack([bf16_bits(dec[(b, l)]["k_new"][t])[sh.kv_heads] for b in range(w.batch)])
                vn = np.stack([bf16_bits(dec[(b, l)]["v_new"][t])[sh.kv_heads] for b in range(w.batch)])
                outs.append(o.decode_layer(l, q, kn, vn))
            # the exchange: one all-reduce of [batch][layers][C_max] partial sums, then every shard takes the sums
            C_max = max(o.dims(b)[2] for b in range(w.batch))
            buf = torch.zeros((w.batch, w.n_layers, C_max), dtype=torch.float64)
            for b in range(w.batch):
                for l in range(w.n_layers):
                    sc = o.chunk_scores(b, l)
                    buf[b, l, :len(sc)] = torch.from_numpy(sc)
            dist.all_reduce(buf)
            scores = {}
            for b in range(w.batch):
                for l in range(w.n_layers):
                    C = o.dims(b)[2]
                    scores[(b, l)] = buf[b, l, :C].numpy().copy()
                    o.set_chunk_scores(b, l, scores[(b, l)])
            o.step_end()
            trace.append({"out": outs, "scores": scores,
                          "sel": {(b, l): o.selected(b, l).tolist() for b in range(w.batch) for l in range(w.n_layers)},
                          "tab": {(b, l): [x.tolist() for x in o.residency(b, l)] for b in range(w.batch) for l in range(w.n_layers)}})
        out[rank] = (sh.q_heads, sh.roles.tolist(), trace)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("split_anchors", [False, True])
def test_two_head_shards_equal_one_oracle(split_anchors):
    world, seed = 2, 13
    w = _workload(split_anchors)
    ref = _run_reference(w, seed)
    port = 21000 + os.getpid() % 4000 + (1 if split_anchors else 0)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, split_anchors, seed, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in (0, 1):
        q_heads, roles, trace = res[r]
        roles = np.array(roles)
        for t, (got, want) in enumerate(zip(trace, ref)):
            for l in range(w.n_layers):
                assert np.array_equal(got["out"][l], want["out"][l][:, q_heads]), (r, t, l)       # a head's attention is its own
                has_anchor_somewhere = (w.roles[l] == A).any()
                for b in range(w.batch):
                    if has_anchor_somewhere:
                        if split_anchors:
                            assert np.abs(got["scores"][(b, l)] - want["scores"][(b, l)]).max() < 1e-12
                        else:
                            assert np.array_equal(got["scores"][(b, l)], want["scores"][(b, l)])
                    if (roles[l] == T).any():                                                     # the shard has a tidal table in this layer
                        assert got["sel"][(b, l)] == want["sel"][(b, l)], (r, t, l, b)
                        assert got["tab"][(b, l)] == want["tab"][(b, l)], (r, t, l, b)


def test_shard_plan_keeps_groups_together_and_flags_anchor_layers():
    sys.path.insert(0, ROOT)
    from paper_2608_22704_b200.sharded import shard_plan
    roles = np.array([[A, T, T, F], [T, F, T, T], [F, T, A, T]], np.uint8)
    plan = shard_plan(roles, 8, 2)
    assert [s.kv_heads for s in plan] == [[0, 1], [2, 3]]
    assert [s.q_heads for s in plan] == [[0, 1, 2, 3], [4, 5, 6, 7]]
    assert plan[1].roles.tolist() == [[T, F], [T, T], [A, T]]
    assert plan[0].global_anchor_layers.tolist() == plan[1].global_anchor_layers.tolist() == [1, 0, 1]
    with pytest.raises(ValueError):
        shard_plan(roles, 8, 3)
