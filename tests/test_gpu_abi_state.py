"""Call-order and capacity errors of the C ABI on a real device: every misuse returns a status, nothing faults (needs a B200)."""
import numpy as np
import pytest
import torch

from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, tiny_custom

pytestmark = pytest.mark.gpu


def _mk(wnw, w, **kw):
    return wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(w.audio_lens), w.text_capacity,
                          w.chunk, w.budget, w.roles, topk=w.topk, **kw)


def _place(wnw, h, syn, b, layers):
    for l in layers:
        p = syn.prefill(b, l)
        dev = torch.device("cuda:0")
        wnw.wnw_place_prefill(h, b, l, p["k"].to(dev), p["v"].to(dev), p["audio_begin"], p["audio_end"], p["q_last"].to(dev))


def test_call_order_and_capacity_errors():
    import paper_2608_22704_b200 as wnw
    dev = torch.device("cuda:0")
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=4, audio_lens=(64, 64), chunk=16, n_steps=2)
    syn = Synth(w, seed=1)
    h = _mk(wnw, w)
    try:
        q = torch.zeros((1, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        kn = torch.zeros((1, w.n_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        out = torch.zeros_like(q)

        def expect(status, fn, *a, **k):
            with pytest.raises(wnw.WnwError) as e:
                fn(*a, **k)
            assert e.value.status == status, e.value

        expect(wnw.WNW_ERR_STATE, wnw.wnw_step_begin, h, [0])                       # decode before prefill
        expect(wnw.WNW_ERR_STATE, wnw.wnw_get_seq_dims, h, 0)
        _place(wnw, h, syn, 0, [0])
        expect(wnw.WNW_ERR_STATE, wnw.wnw_step_begin, h, [0])                       # only one of two layers placed
        p = syn.prefill(0, 0)
        expect(wnw.WNW_ERR_STATE, wnw.wnw_place_prefill, h, 0, 1, p["k"][:-1].to(dev), p["v"][:-1].to(dev), p["audio_begin"],
               p["audio_end"] - 1, p["q_last"].to(dev))                            # token counts differ from layer 0
        _place(wnw, h, syn, 0, [1])
        expect(wnw.WNW_ERR_INVALID_ARG, wnw.wnw_step_begin, h, [0, 0])              # duplicate sequence
        expect(wnw.WNW_ERR_INVALID_ARG, wnw.wnw_step_begin, h, [5])
        expect(wnw.WNW_ERR_STATE, wnw.wnw_decode_layer, h, 0, q, kn, kn, out)       # no step open
        wnw.wnw_step_begin(h, [0])
        expect(wnw.WNW_ERR_STATE, wnw.wnw_step_begin, h, [0])                       # step already open
        expect(wnw.WNW_ERR_STATE, wnw.wnw_decode_layer, h, 1, q, kn, kn, out)       # layers out of order
        expect(wnw.WNW_ERR_STATE, wnw.wnw_decode_layer_full, h, 0, q, kn, kn, out)  # tiered cache, full-cache entry point
        expect(wnw.WNW_ERR_INVALID_ARG, wnw.wnw_decode_layer, h, 0, q, kn, None, out)
        expect(wnw.WNW_ERR_STATE, wnw.wnw_step_end, h)                              # not all layers done
        expect(wnw.WNW_ERR_STATE, wnw.wnw_place_prefill, h, 1, 0, p["k"].to(dev), p["v"].to(dev), p["audio_begin"],
               p["audio_end"], p["q_last"].to(dev))                                # placement inside a step
        wnw.wnw_decode_layer(h, 0, q, kn, kn, out)
        expect(wnw.WNW_ERR_STATE, wnw.wnw_decode_layer, h, 1, q, None, None, out)   # append in layer 0 but not in layer 1
        wnw.wnw_decode_layer(h, 1, q, kn, kn, out)
        wnw.wnw_step_end(h)
        wnw.wnw_step_begin(h, [0]); wnw.wnw_decode_layer(h, 0, q, kn, kn, out); wnw.wnw_decode_layer(h, 1, q, kn, kn, out)
        wnw.wnw_step_end(h)                                                        # text capacity (4 + 2 steps) is now full
        wnw.wnw_step_begin(h, [0])
        expect(wnw.WNW_ERR_CAPACITY, wnw.wnw_decode_layer, h, 0, q, kn, kn, out)
        wnw.wnw_decode_layer(h, 0, q, None, None, out)                             # attending without appending still works
        wnw.wnw_decode_layer(h, 1, q, None, None, out)
        wnw.wnw_step_end(h)
        wnw.wnw_sync(h)                                                            # no sticky device-side error
        assert wnw.wnw_get_seq_dims(h, 0)[1] == 6
        big = torch.zeros((200, w.n_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        expect(wnw.WNW_ERR_CAPACITY, wnw.wnw_place_prefill, h, 1, 0, big, big, 10, 190, p["q_last"].to(dev))   # audio > capacity
        expect(wnw.WNW_ERR_INVALID_ARG, wnw.wnw_graph_begin, h, [0], None)          # the default stream cannot be captured
        expect(wnw.WNW_ERR_STATE, wnw.wnw_graph_launch, h, torch.cuda.Stream())     # nothing captured yet
    finally:
        wnw.wnw_destroy(h)


def test_replacing_a_sequence_invalidates_the_captured_graph():
    import paper_2608_22704_b200 as wnw
    dev = torch.device("cuda:0")
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=4, audio_lens=(64,), chunk=16, n_steps=8)
    syn = Synth(w, seed=2)
    h = _mk(wnw, w)
    try:
        _place(wnw, h, syn, 0, [0, 1])
        st = torch.cuda.Stream()
        q = torch.zeros((1, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        kn = torch.zeros((1, w.n_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        out = torch.zeros_like(q)
        torch.cuda.synchronize()
        wnw.wnw_graph_begin(h, [0], st)
        wnw.wnw_step_begin(h, [0])
        for l in range(2):
            wnw.wnw_decode_layer(h, l, q, kn, kn, out, stream=st)
        wnw.wnw_step_end(h, stream=st)
        wnw.wnw_graph_end(h, st)
        assert wnw.wnw_get_seq_dims(h, 0)[1] == 4                                  # capture ran nothing
        wnw.wnw_graph_launch(h, st); wnw.wnw_graph_launch(h, st)
        wnw.wnw_sync(h)
        assert wnw.wnw_get_seq_dims(h, 0)[1] == 6
        assert wnw.wnw_get_stats(h)["steps"] == 2
        _place(wnw, h, syn, 0, [0, 1])                                             # re-place: work lists are rebuilt
        with pytest.raises(wnw.WnwError) as e:
            wnw.wnw_graph_launch(h, st)
        assert e.value.status == wnw.WNW_ERR_STATE
    finally:
        wnw.wnw_destroy(h)


@pytest.mark.parametrize("mode", [1, 2])
def test_layer_dependency_modes_give_identical_results(mode):
    """Chained layers (the kernel waits for the preceding work before it reads q/k_new/v_new) and plain serial launches
    stay in lock-step with the oracle, eagerly and under graph replay, and agree with the default overlapped launches up
    to the rounding order of the split merge (the work is cut differently per mode); selections and tables are equal."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    from workloads import ROLE_ANCHOR as A, ROLE_FIXED as F, ROLE_TIDAL as T, tiny_custom
    w = tiny_custom(n_layers=5, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=8, audio_lens=(640, 300), chunk=32, budget=0.2,
                    n_steps=8, roles=[[A, T, T, F], [T, F, T, F], [A, T, F, T], [T, T, F, F], [A, A, T, F]], region=32,
                    jump_every=3)
    ref, ls = Lockstep(w, seed=8), Lockstep(w, seed=8)
    try:
        wnw.wnw_set_layer_dependency(ls.h, mode)
        ref.prefill(); ls.prefill()
        for t in range(8):
            a = ref.decode_step(t, graph=t >= 2)
            b = ls.decode_step(t, graph=t >= 2)
            for (_, _, _, oa), (_, _, _, ob) in zip(a, b):
                assert (oa.float() - ob.float()).abs().max().item() <= 2e-2
            for bb in range(w.batch):
                for l in range(w.n_layers):
                    if (w.roles[l] == ROLE_TIDAL).any():
                        ta, tb = wnw.wnw_get_residency(ref.h, bb, l), wnw.wnw_get_residency(ls.h, bb, l)
                        assert np.array_equal(ta[0], tb[0]) and np.array_equal(ta[1], tb[1])
        ls.check_stats()
    finally:
        ref.close(); ls.close()


def test_layer_dependency_rejects_bad_mode():
    import paper_2608_22704_b200 as wnw
    from workloads import config0
    w = config0()
    h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, 1024, w.text_capacity, w.chunk, w.budget,
                       w.roles, topk=w.topk)
    try:
        with pytest.raises(wnw.WnwError):
            wnw.wnw_set_layer_dependency(h, 4)
        wnw.wnw_set_layer_dependency(h, 1)
    finally:
        wnw.wnw_destroy(h)


def test_bounded_wait_runs_out_and_reports_timeout():
    """The tidal CTAs of a replayed step wait (bounded, about a second of SM clocks) for the recall epoch of the previous
    step.  With the expected epoch pushed beyond anything that will be published the waits run out: the kernels finish,
    wnw_sync reports WNW_ERR_TIMEOUT, nothing hangs, and the context stays usable."""
    import time
    import paper_2608_22704_b200 as wnw
    dev = torch.device("cuda:0")
    A, T, F = ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=4, audio_lens=(200,), chunk=16, budget=0.25,
                    n_steps=6, roles=[[A, T], [A, T]])
    syn = Synth(w, seed=1)

    def run(h, n_replays, skew_before=None):
        _place(wnw, h, syn, 0, range(w.n_layers))
        dec = [syn.decode(0, l) for l in range(w.n_layers)]
        sq = torch.zeros((w.n_layers, 1, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        skn = torch.zeros((w.n_layers, 1, w.n_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
        svn, out = torch.zeros_like(skn), torch.zeros_like(sq)
        st = torch.cuda.Stream(device=dev)
        torch.cuda.synchronize()
        wnw.wnw_graph_begin(h, [0], st)
        wnw.wnw_step_begin(h, [0])
        for l in range(w.n_layers):
            wnw.wnw_decode_layer(h, l, sq[l], skn[l], svn[l], out[l], stream=st)
        wnw.wnw_step_end(h, stream=st)
        wnw.wnw_graph_end(h, st)
        for t in range(n_replays):
            if skew_before == t:
                wnw.wnw_debug_advance_step_epoch(h, 3)
            with torch.cuda.stream(st):
                for l in range(w.n_layers):
                    sq[l, 0].copy_(dec[l]["q"][t]); skn[l, 0].copy_(dec[l]["k_new"][t]); svn[l, 0].copy_(dec[l]["v_new"][t])
                wnw.wnw_graph_launch(h, st)
        return out

    h = _mk(wnw, w)
    try:
        run(h, 2)
        wnw.wnw_sync(h)                                  # healthy replays: no status
    finally:
        wnw.wnw_destroy(h)
    h = _mk(wnw, w)
    try:
        t0 = time.perf_counter()
        run(h, 3, skew_before=2)
        with pytest.raises(wnw.WnwError) as e:
            wnw.wnw_sync(h)
        elapsed = time.perf_counter() - t0
        assert e.value.status == wnw.WNW_ERR_TIMEOUT
        assert 0.3 < elapsed < 30.0                      # the waits gave up by themselves
    finally:
        wnw.wnw_destroy(h)
    h = _mk(wnw, w)                                      # the context is still good
    try:
        out = run(h, 2)
        wnw.wnw_sync(h)
        assert torch.isfinite(out.float()).all()
    finally:
        wnw.wnw_destroy(h)
