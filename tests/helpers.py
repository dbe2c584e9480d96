"""Shared test helpers: bf16 bit conversion, a numpy dense attention used to pin the oracle, oracle set-up."""
from __future__ import annotations

import numpy as np

from workloads import Synth, Workload
from workloads.synth import bf16_bits


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dense_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float, mask: np.ndarray | None = None):
    """Textbook softmax attention in float64.  q [d], K,V [n,d], mask [n] bool (True = visible).
    Returns (out [d], p [n])."""
    logits = (K @ q) * scale
    if mask is not None:
        logits = np.where(mask, logits, -np.inf)
    if not np.isfinite(logits).any():
        return np.zeros(V.shape[1]), np.zeros(len(logits))
    e = np.exp(logits - logits[np.isfinite(logits)].max())
    p = e / e.sum()
    return p @ V, p


def make_oracle(w: Workload, budget: float | None = None, max_batch: int | None = None, score_scope: int = 0,
                residency: int = 0, evict_lag: int = 3):
    from oracle.wnw_oracle import Oracle
    return Oracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, max_batch or w.batch, max(max(w.audio_lens), 1),
                  w.text_capacity, w.chunk, w.topk, w.budget if budget is None else budget, w.roles, score_scope=score_scope,
                  residency=residency, evict_lag=evict_lag)


def place_all(oracle, syn: Synth, keep: bool = False):
    """Place every (seq, layer) prefill into the oracle.  With keep=True also returns the float64 K,V per (seq, layer)."""
    w = syn.w
    kept = {}
    for b in range(w.batch):
        for l in range(w.n_layers):
            p = syn.prefill(b, l)
            kb, vb, qb = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_last"])
            oracle.place_prefill(b, l, kb, vb, p["audio_begin"], p["audio_end"], qb)
            if keep:
                kept[(b, l)] = (bf16_bits_to_f64(kb), bf16_bits_to_f64(vb), bf16_bits_to_f64(qb), p["audio_begin"], p["audio_end"])
    return kept
