"""Seeded synthetic workloads shaped like the paper's long-form speech decoding.

The paper measures on speech corpora with trained 3B backbones; neither is
available, so these inputs take the *shapes* of those runs (layers, GQA heads,
head_dim, audio length = minutes x frame rate; Notation paragraph of the Method
section) and the *structure* the paper reports for attention over audio: a
prefill-time attention sink on the first audio positions and a decode-time
focus that sweeps through the clip (Prefill-Decode Attention Mismatch
subsection).  They stand in for the paper's datasets.

Recipe, per (sequence, layer, KV-head), all N(0,1) draws from a torch generator
seeded by (seed, tag, sequence, layer):
  * sink direction  s   = unit vector,      region codes e_r = unit vectors,
    one per region of `region` consecutive audio tokens;
  * V ~ N(0,1);  text K ~ N(0,1);
    audio K_tau = N(0,I) + 4 e_{tau // region} + [tau < 4] 4 s;
  * decode query of step t (every q-head of the group):
      q_t = N(0,I) + (sqrt(d)/2) s + 1.5 sqrt(d) sum_r w_r(t) e_r,
      w_r(t) = exp(-(r + 1/2 - c_t/region)^2 / 2),
    with focus centre c_t = (t / n_steps) T_a (drift), or, for the
    recall-stress workload, c_t redrawn uniformly every `jump_every` steps;
  * prefill query q_last = N(0,I) + 2 sqrt(d) s   (sink dominated);
  * k_new, v_new ~ N(0,1) per decode step.
Everything is rounded to bf16 once; the same bits go to every consumer.

This module draws numbers and describes shapes.  It contains no attention,
scoring, selection or residency logic.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np
import torch

ROLE_ANCHOR = 0
ROLE_TIDAL = 1
ROLE_FIXED = 2

_TAG_DIRS, _TAG_PREFILL, _TAG_DECODE, _TAG_CENTRE, _TAG_ROLES, _TAG_LENS, _TAG_PREFILL_Q = 1, 2, 3, 4, 5, 6, 7


@dataclass
class Workload:
    """Shape description of one synthetic decoding job."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_text: int                 # text prefix tokens (before the audio)
    audio_lens: List[int]       # per sequence
    chunk: int                  # tokens per (non-overlapping) chunk
    budget: float               # fraction of audio chunks a non-anchor head keeps on GPU
    n_steps: int                # decode steps
    roles: np.ndarray           # uint8 [n_layers, n_kv_heads]
    topk: int = 3               # chunks selected per step (the paper's k)
    evict_lag: int = 3          # the paper's delta
    region: int = 64            # audio tokens per region code
    jump_every: int = 0         # 0: drifting focus; n>0: focus jumps every n steps
    sweep_steps: int = 0        # steps for one sweep of the clip (0: n_steps)
    n_prefill_queries: int = 1  # text queries whose attention ranks the audio at prefill (1: the last prefix query only)

    @property
    def batch(self) -> int:
        return len(self.audio_lens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def text_capacity(self) -> int:
        return self.n_text + self.n_steps

    def n_chunks(self, seq: int) -> int:
        return -(-self.audio_lens[seq] // self.chunk)


def paper_chunk_geometry(window_s: float, stride_s: float, tokens_per_s: float):
    """Tokens per chunk and per segment for a chunk window and stride in seconds at an audio frame rate
    ("Chunk Structure": n_c = ceil(W_c r_tok), n_s = ceil(W_s r_tok))."""
    return math.ceil(window_s * tokens_per_s), math.ceil(stride_s * tokens_per_s)


def _mix(seed: int, tag: int, a: int = 0, b: int = 0) -> int:
    x = (seed + 1) * 0x9E3779B97F4A7C15 + tag * 0xBF58476D1CE4E5B9 + a * 0x94D049BB133111EB + b * 0xD6E8FEB86659FD93
    x ^= x >> 31
    return x % (2 ** 62)


def _roles_cfg1(n_layers: int, seed: int) -> np.ndarray:
    rs = np.random.RandomState(_mix(seed, _TAG_ROLES) % (2 ** 31))
    base = np.array([ROLE_ANCHOR] + [ROLE_TIDAL] * 5 + [ROLE_FIXED] * 2, dtype=np.uint8)
    return np.stack([base[rs.permutation(8)] for _ in range(n_layers)])


def _roles_cfg2(n_layers: int, n_kv: int, seed: int) -> np.ndarray:
    rs = np.random.RandomState(_mix(seed, _TAG_ROLES, 2) % (2 ** 31))
    u = rs.random_sample((n_layers, n_kv))
    roles = np.where(u < 1 / 8, ROLE_ANCHOR, np.where(u < 5 / 8, ROLE_TIDAL, ROLE_FIXED)).astype(np.uint8)
    for blk in range(0, n_layers, 4):
        sub = roles[blk:blk + 4]
        if not (sub == ROLE_ANCHOR).any():
            l = blk + rs.randint(0, sub.shape[0])
            roles[l, rs.randint(0, n_kv)] = ROLE_ANCHOR
    return roles


def config0(seed: int = 0) -> Workload:
    """Tiny single layer: 8q/4kv heads, d=64, roles {anchor, tidal, tidal, fixed}."""
    roles = np.array([[ROLE_ANCHOR, ROLE_TIDAL, ROLE_TIDAL, ROLE_FIXED]], dtype=np.uint8)
    return Workload("cfg0_tiny", 1, 8, 4, 64, 32, [1024], 32, 0.2, 16, roles, region=32)


def config1(seed: int = 0, n_steps: int = 256) -> Workload:
    """3B stack shaped like Voxtral-mini-3b: 30 layers, 32q/8kv, d=128, 4 min of audio at 12.5 tok/s."""
    w = Workload("cfg1_voxtral3b_4min", 30, 32, 8, 128, 64, [3000], 64, 0.2, n_steps, _roles_cfg1(30, seed))
    w.sweep_steps = 256
    return w


def config2(seed: int = 0, n_steps: int = 512) -> Workload:
    """3B stack shaped like Qwen2.5-Omni-3B: 36 layers, 16q/2kv, d=128, 10 min at 25 tok/s."""
    w = Workload("cfg2_qwen_omni3b_10min", 36, 16, 2, 128, 64, [15000], 64, 0.2, n_steps, _roles_cfg2(36, 2, seed))
    w.sweep_steps = 512
    return w


def config3(seed: int = 0, batch: int = 32, n_steps: int = 128) -> Workload:
    """Batched serving: config-1 shapes, ragged audio lengths U{2000..7500}."""
    rs = np.random.RandomState(_mix(seed, _TAG_LENS) % (2 ** 31))
    lens = [int(x) for x in rs.randint(2000, 7501, size=batch)]
    w = Workload("cfg3_batched_ragged", 30, 32, 8, 128, 64, lens, 64, 0.2, n_steps, _roles_cfg1(30, seed))
    w.sweep_steps = 128
    return w


def config4(seed: int = 0, budget: float = 0.2, chunk: int = 64, batch: int = 8, n_steps: int = 64) -> Workload:
    """Recall stress: config-1 shapes, 7500 audio tokens, focus jumps every 4 steps."""
    w = Workload(f"cfg4_recall_b{int(round(budget * 100))}_c{chunk}", 30, 32, 8, 128, 64, [7500] * batch, chunk,
                 budget, n_steps, _roles_cfg1(30, seed), jump_every=4)
    return w


def tiny_custom(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_text=5, audio_lens=(100,), chunk=16,
                budget=0.25, n_steps=6, roles=None, topk=3, region=16, jump_every=0, name="tiny") -> Workload:
    """Small free-form workload for tests (ragged tails, odd sizes, several sequences)."""
    if roles is None:
        pattern = [ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED, ROLE_TIDAL]
        roles = np.array([[pattern[(l + h) % 4] for h in range(n_kv_heads)] for l in range(n_layers)], dtype=np.uint8)
        roles[0, 0] = ROLE_ANCHOR
    return Workload(name, n_layers, n_q_heads, n_kv_heads, head_dim, n_text, list(audio_lens), chunk, budget,
                    n_steps, np.asarray(roles, dtype=np.uint8), topk=topk, region=region, jump_every=jump_every)


class Synth:
    """Draws the tensors of a Workload.  All outputs are torch.bfloat16 on `device`."""

    def __init__(self, workload: Workload, seed: int = 0, device: str = "cpu"):
        self.w = workload
        self.seed = seed
        self.device = torch.device(device)
        self._dirs: Dict[Tuple[int, int], Tuple[torch.Tensor, torch.Tensor]] = {}

    # -- helpers ---------------------------------------------------------
    def _gen(self, tag: int, seq: int, layer: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed(_mix(self.seed, tag, seq, layer))
        return g

    def _randn(self, g: torch.Generator, *shape: int) -> torch.Tensor:
        return torch.randn(*shape, generator=g, device=self.device, dtype=torch.float32)

    def n_regions(self, seq: int) -> int:
        return max(1, -(-self.w.audio_lens[seq] // self.w.region))

    def dirs(self, seq: int, layer: int) -> Tuple[torch.Tensor, torch.Tensor]:
        """(s [Hkv,d], e [Hkv,n_regions,d]) unit directions, fp32."""
        key = (seq, layer)
        if key not in self._dirs:
            g = self._gen(_TAG_DIRS, seq, layer)
            w = self.w
            s = self._randn(g, w.n_kv_heads, w.head_dim)
            e = self._randn(g, w.n_kv_heads, self.n_regions(seq), w.head_dim)
            s = s / s.norm(dim=-1, keepdim=True)
            e = e / e.norm(dim=-1, keepdim=True)
            self._dirs[key] = (s, e)
        return self._dirs[key]

    def centres(self, seq: int) -> np.ndarray:
        """Focus centre c_t (audio position) for every decode step, float64 [n_steps]."""
        w = self.w
        T_a = w.audio_lens[seq]
        t = np.arange(w.n_steps, dtype=np.float64)
        if w.jump_every > 0:
            rs = np.random.RandomState(_mix(self.seed, _TAG_CENTRE, seq) % (2 ** 31))
            draws = rs.random_sample(-(-w.n_steps // w.jump_every)) * T_a
            return np.repeat(draws, w.jump_every)[:w.n_steps]
        sweep = w.sweep_steps if w.sweep_steps > 0 else w.n_steps
        return (t / sweep) * T_a

    # -- tensors ---------------------------------------------------------
    def prefill(self, seq: int, layer: int) -> dict:
        """Prefill K,V [n_tokens,Hkv,d] (text prefix then audio) and the last prefix query [Hq,d]."""
        w = self.w
        T_a = w.audio_lens[seq]
        n = w.n_text + T_a
        g = self._gen(_TAG_PREFILL, seq, layer)
        s, e = self.dirs(seq, layer)
        k = self._randn(g, n, w.n_kv_heads, w.head_dim)
        v = self._randn(g, n, w.n_kv_heads, w.head_dim)
        if T_a > 0:
            region_of = torch.arange(T_a, device=self.device) // w.region        # [T_a]
            code = e[:, region_of, :].permute(1, 0, 2)                           # [T_a,Hkv,d]
            k[w.n_text:] += 4.0 * code
            n_sink = min(4, T_a)
            k[w.n_text:w.n_text + n_sink] += 4.0 * s.unsqueeze(0)
        q_noise = self._randn(g, w.n_q_heads, w.head_dim)
        s_q = s.repeat_interleave(w.group, dim=0)                                # [Hq,d]
        q_last = q_noise + 2.0 * math.sqrt(w.head_dim) * s_q
        out = {"k": k.to(torch.bfloat16).contiguous(), "v": v.to(torch.bfloat16).contiguous(),
               "q_last": q_last.to(torch.bfloat16).contiguous(),
               "n_tokens": n, "audio_begin": w.n_text, "audio_end": n}
        if w.n_prefill_queries > 1:
            # earlier text queries: each leans on the sink and on one region of its own; the last one is q_last
            gq = self._gen(_TAG_PREFILL_Q, seq, layer)
            m = w.n_prefill_queries - 1
            qn = self._randn(gq, m, w.n_q_heads, w.head_dim)
            n_reg = max(self.n_regions(seq), 1)
            reg = torch.randint(0, n_reg, (m,), generator=gq, device=self.device)
            lean = e[:, reg, :].permute(1, 0, 2).repeat_interleave(w.group, dim=1) if T_a > 0 else torch.zeros_like(qn)
            qn = qn + 1.0 * math.sqrt(w.head_dim) * s_q.unsqueeze(0) + 1.0 * math.sqrt(w.head_dim) * lean
            out["q_text"] = torch.cat([qn, q_last.unsqueeze(0)], dim=0).to(torch.bfloat16).contiguous()
        return out

    def decode(self, seq: int, layer: int) -> dict:
        """Decode inputs of every step: q [n_steps,Hq,d], k_new, v_new [n_steps,Hkv,d]."""
        w = self.w
        g = self._gen(_TAG_DECODE, seq, layer)
        s, e = self.dirs(seq, layer)
        d = w.head_dim
        q = self._randn(g, w.n_steps, w.n_q_heads, d)
        k_new = self._randn(g, w.n_steps, w.n_kv_heads, d)
        v_new = self._randn(g, w.n_steps, w.n_kv_heads, d)
        c = torch.from_numpy(self.centres(seq)).to(self.device)                  # [n_steps] f64
        r = torch.arange(self.n_regions(seq), device=self.device, dtype=torch.float64)
        wts = torch.exp(-0.5 * (r.unsqueeze(0) + 0.5 - c.unsqueeze(1) / w.region) ** 2).to(torch.float32)
        focus = torch.einsum("tr,hrd->thd", wts, e)                              # [n_steps,Hkv,d]
        bias = 0.5 * math.sqrt(d) * s.unsqueeze(0) + 1.5 * math.sqrt(d) * focus  # [n_steps,Hkv,d]
        q = q + bias.repeat_interleave(w.group, dim=1)
        return {"q": q.to(torch.bfloat16).contiguous(), "k_new": k_new.to(torch.bfloat16).contiguous(),
                "v_new": v_new.to(torch.bfloat16).contiguous()}


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw bf16 bit patterns of a bf16 tensor as a host uint16 array (same shape)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
