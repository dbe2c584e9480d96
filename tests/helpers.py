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


# ---- FP8 (e4m3) storage of the tidal tier: what the stored rows decode to -------------------------------------------
# The library may keep the tidal heads' audio K,V as e4m3 bytes with one power-of-two scale per (chunk, head, K|V)
# (KV quantisation is orthogonal to the method: Baselines paragraph, footnote on KV quantisation).  The oracle knows
# nothing of storage formats: it is handed the values those bytes decode to, which are exact bf16 numbers, so every
# tolerance stays what it is.  This is the definition of the format, written out in float64.

def e4m3_round(x: np.ndarray) -> np.ndarray:
    """Nearest e4m3 value (4 exponent bits, bias 7, 3 mantissa bits, subnormals, largest finite 448), ties to even;
    |x| beyond 448 saturates.  float64 in, float64 out."""
    x = np.asarray(x, np.float64)
    a = np.abs(x)
    _, e = np.frexp(a)                                  # a = m * 2^e, m in [0.5, 1)
    binade = np.maximum(e - 1, -6)                      # below 2^-6 the subnormals share the smallest binade's spacing
    step = np.ldexp(1.0, binade - 3)
    q = np.minimum(np.rint(a / step) * step, 448.0)     # np.rint rounds ties to even
    return np.copysign(q, x)


def fp8_scale_exponent(absmax: float) -> int:
    """The power of two e with absmax / 2^e in (224, 448]: the largest magnitude of the block lands in e4m3's top binade."""
    if absmax == 0.0:
        return 0
    m, e = np.frexp(absmax)                             # absmax = m * 2^e, m in [0.5, 1)  ->  1.m' * 2^(e-1)
    return int(e - 1 - 8 + (1 if m > 0.875 else 0))     # 448 = 1.75 * 2^8


def dequantised_tidal_bits(kb: np.ndarray, vb: np.ndarray, roles_l: np.ndarray, audio_begin: int, audio_end: int, chunk: int):
    """bf16 bit patterns [n_tokens][n_kv_heads][d] of one layer's prefix with the audio rows of the tidal heads replaced
    by what their e4m3 storage decodes to (scale per chunk, head and K|V from the chunk's largest magnitude)."""
    from workloads import ROLE_TIDAL
    out = []
    for bits in (kb, vb):
        bits = np.array(bits, dtype=np.uint16, copy=True)
        for h in np.nonzero(np.asarray(roles_l) == ROLE_TIDAL)[0]:
            for c0 in range(audio_begin, audio_end, chunk):
                c1 = min(c0 + chunk, audio_end)
                x = bf16_bits_to_f64(bits[c0:c1, h])
                e = fp8_scale_exponent(float(np.abs(x).max()))
                deq = np.ldexp(e4m3_round(np.ldexp(x, -e)), e).astype(np.float32)
                u = deq.view(np.uint32)
                assert not (u & 0xFFFF).any()            # three mantissa bits and a power-of-two scale: exact in bf16
                bits[c0:c1, h] = (u >> 16).astype(np.uint16)
        out.append(bits)
    return out[0], out[1]
