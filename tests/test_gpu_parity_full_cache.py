"""The full-cache comparison path (the "Full Cache" baseline of the Baselines paragraph) against the CPU oracle.

An oracle whose KV heads are all anchors attends to text + all audio for every head, which is exactly what
wnw_decode_layer_full computes; the oracle's attention is itself pinned to numpy dense attention by the CPU tests.
Every way the step can be issued is compared element by element: eager and replayed from a captured graph, one launch
per layer (independent, chained, serial) and all layers in one launch, with and without appends, ragged batches and
every query-group size the kernel has a code path for.  Needs a B200."""
import numpy as np
import pytest
import torch

import paper_2608_22704_b200 as wnw
from helpers import bf16_bits_to_f64
from oracle.wnw_oracle import Oracle
from workloads import Synth, config1, tiny_custom
from workloads.synth import bf16_bits

pytestmark = pytest.mark.gpu
OUT_TOL = 2e-2


class FullLockstep:
    """A FULL-mode cache and an all-anchor oracle fed the same bits."""

    def __init__(self, w, seed=0, dependency=wnw.WNW_LAYERS_INDEPENDENT, gen_device="cpu"):
        self.w = w
        self.dev = torch.device("cuda:0")
        self.syn = Synth(w, seed=seed, device=gen_device)
        anchors = np.zeros((w.n_layers, w.n_kv_heads), np.uint8)
        self.o = Oracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(max(w.audio_lens), 1), w.text_capacity,
                        w.chunk, w.topk, 1.0, anchors)
        self.h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max(max(w.audio_lens), 0),
                                w.text_capacity, w.chunk, w.budget, w.roles, topk=w.topk, mode=wnw.WNW_MODE_FULL)
        wnw.wnw_set_layer_dependency(self.h, dependency)
        self.dec = {}
        self.max_err = 0.0
        self.graph = None

    def close(self):
        if self.h:
            wnw.wnw_destroy(self.h); self.h = None
        self.o.close()

    def prefill(self):
        w = self.w
        for b in range(w.batch):
            for l in range(w.n_layers):
                p = self.syn.prefill(b, l)
                wnw.wnw_place_prefill(self.h, b, l, p["k"].to(self.dev), p["v"].to(self.dev), p["audio_begin"], p["audio_end"], None)
                torch.cuda.synchronize(self.dev)
                self.o.place_prefill(b, l, bf16_bits(p["k"]), bf16_bits(p["v"]), p["audio_begin"], p["audio_end"],
                                     bf16_bits(p["q_last"]))   # (unused: no head ranks chunks)
        wnw.wnw_sync(self.h)

    def _dec(self, b, l):
        if (b, l) not in self.dec:
            self.dec[(b, l)] = self.syn.decode(b, l)
        return self.dec[(b, l)]

    def step(self, t, active=None, append=True, graph=False):
        w = self.w
        active = list(range(w.batch)) if active is None else list(active)
        qs = [torch.stack([self._dec(b, l)["q"][t] for b in active]).to(self.dev) for l in range(w.n_layers)]
        kns = [torch.stack([self._dec(b, l)["k_new"][t] for b in active]).to(self.dev) if append else None for l in range(w.n_layers)]
        vns = [torch.stack([self._dec(b, l)["v_new"][t] for b in active]).to(self.dev) if append else None for l in range(w.n_layers)]
        if graph:
            if self.graph is None:
                self.gs = torch.cuda.Stream(device=self.dev)
                self.gq = [torch.empty_like(x) for x in qs]
                self.gk = [torch.empty_like(x) if x is not None else None for x in kns]
                self.gv = [torch.empty_like(x) if x is not None else None for x in vns]
                self.gout = [torch.empty_like(x) for x in qs]
                torch.cuda.synchronize(self.dev)
                wnw.wnw_graph_begin(self.h, active, self.gs)
                wnw.wnw_step_begin(self.h, active)
                for l in range(w.n_layers):
                    wnw.wnw_decode_layer_full(self.h, l, self.gq[l], self.gk[l], self.gv[l], self.gout[l], stream=self.gs)
                wnw.wnw_step_end(self.h, stream=self.gs)
                wnw.wnw_graph_end(self.h, self.gs)
                self.graph = True
            self.gs.wait_stream(torch.cuda.current_stream(self.dev))
            with torch.cuda.stream(self.gs):
                for l in range(w.n_layers):
                    self.gq[l].copy_(qs[l])
                    if append:
                        self.gk[l].copy_(kns[l]); self.gv[l].copy_(vns[l])
                    self.gout[l].fill_(float("nan"))
            wnw.wnw_graph_launch(self.h, self.gs)
            self.gs.synchronize()
            outs = self.gout
        else:
            outs = [torch.full_like(x, float("nan")) for x in qs]
            wnw.wnw_step_begin(self.h, active)
            for l in range(w.n_layers):
                wnw.wnw_decode_layer_full(self.h, l, qs[l], kns[l], vns[l], outs[l])
            wnw.wnw_step_end(self.h)
        wnw.wnw_sync(self.h)
        self.o.step_begin(active)
        for l in range(w.n_layers):
            ref = self.o.decode_layer(l, bf16_bits(qs[l].cpu()), bf16_bits(kns[l].cpu()) if append else None,
                                      bf16_bits(vns[l].cpu()) if append else None)
            got = bf16_bits_to_f64(bf16_bits(outs[l].cpu()))
            assert np.isfinite(got).all(), f"step {t} layer {l}: output not written everywhere"
            err = float(np.abs(got - ref).max())
            self.max_err = max(self.max_err, err)
            assert err <= OUT_TOL, f"full-cache output step {t} layer {l}: max abs err {err:.4f}"
        self.o.step_end()


DEPS = [wnw.WNW_LAYERS_INDEPENDENT, wnw.WNW_LAYERS_CHAINED, wnw.WNW_LAYERS_SERIAL, wnw.WNW_LAYERS_BATCHED]


@pytest.mark.parametrize("dep", DEPS)
@pytest.mark.parametrize("hq,hkv,d", [(2, 2, 64), (8, 2, 128), (16, 2, 128), (32, 2, 64)])   # g = 1, 4, 8, 16
def test_full_cache_matches_oracle_eager_and_replayed(dep, hq, hkv, d):
    """Ragged batch (a clip shorter than a granule, one with a ragged tail, one of many granules), appends every step:
    two eager steps, then replays of a captured step, then an eager step again."""
    w = tiny_custom(n_layers=3, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, n_text=7, audio_lens=(11, 333, 1500), chunk=32,
                    n_steps=8)
    ls = FullLockstep(w, seed=21 + hq, dependency=dep)
    try:
        ls.prefill()
        for t in (0, 1):
            ls.step(t)
        for t in (2, 3, 4, 5):
            ls.step(t, graph=True)
        ls.step(6)
        ls.step(7, graph=True)
        assert ls.max_err > 0
    finally:
        ls.close()


def test_full_cache_without_append_and_subset_of_sequences():
    w = tiny_custom(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=128, n_text=0, audio_lens=(700, 90, 16), chunk=16, n_steps=4)
    ls = FullLockstep(w, seed=5)
    try:
        ls.prefill()
        ls.step(0, append=False)
        ls.step(1, active=[2, 0], append=False)
        ls.step(2, active=[1])
    finally:
        ls.close()


def test_full_cache_text_only_sequence():
    w = tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=40, audio_lens=(0,), chunk=16, n_steps=3)
    ls = FullLockstep(w, seed=6)
    try:
        ls.prefill()
        for t in range(3):
            ls.step(t)
    finally:
        ls.close()


@pytest.mark.parametrize("dep", [wnw.WNW_LAYERS_CHAINED, wnw.WNW_LAYERS_BATCHED])
def test_full_cache_config1_full_size_replayed(dep):
    """Config-1 shapes (30 layers, 32q/8kv, d=128, 3000 audio + 64 text tokens) in the two forms the benchmark times:
    chained layers and all layers in one launch, every step replayed, the oracle following every step."""
    w = config1(n_steps=6)
    ls = FullLockstep(w, seed=0, dependency=dep, gen_device="cuda:0")
    try:
        ls.prefill()
        for t in range(6):
            ls.step(t, graph=True)
    finally:
        ls.close()
