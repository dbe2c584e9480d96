"""ctypes wrapper of the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It never imports the CUDA package.  `build()` compiles
wnw_oracle.c with gcc (-O2, OpenMP over query heads) next to this file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wnw_oracle.c")
_LIB = os.path.join(_HERE, "libwnw_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(C.POINTER(ty))


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.wnwo_create.argtypes = [C.c_int] * 9 + [C.c_double, C.c_double, C.POINTER(C.c_uint8), C.c_int, C.c_int, C.c_int,
                                     C.POINTER(C.c_void_p)]
        _lib.wnwo_create_shard.argtypes = [C.c_int] * 9 + [C.c_double, C.c_double, C.POINTER(C.c_uint8), C.c_int, C.c_int, C.c_int,
                                           C.POINTER(C.c_uint8), C.POINTER(C.c_void_p)]
        _lib.wnwo_set_chunk_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_double)]
        _lib.wnwo_destroy.argtypes = [C.c_void_p]
        _lib.wnwo_destroy.restype = None
        _lib.wnwo_score_source.argtypes = [C.c_void_p, C.c_int]
        _lib.wnwo_place_prefill.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16),
                                            C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint16)]
        _lib.wnwo_place_prefill_multi.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16),
                                                  C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.c_int]
        _lib.wnwo_append_audio.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16), C.c_int]
        _lib.wnwo_step_begin.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.c_int]
        _lib.wnwo_decode_layer.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16),
                                           C.POINTER(C.c_uint16), C.POINTER(C.c_double)]
        _lib.wnwo_step_end.argtypes = [C.c_void_p]
        _lib.wnwo_get_dims.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_int)] * 4
        _lib.wnwo_get_chunk_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_double)]
        _lib.wnwo_get_prefill_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_double)]
        _lib.wnwo_get_selected.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_get_residency.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_longlong)]
        _lib.wnwo_set_residency.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_longlong)]
        _lib.wnwo_get_fixed_set.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_set_fixed_set.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int]
        _lib.wnwo_get_stats.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_longlong)] * 3
        _lib.wnwo_attention_row.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint16),
                                            C.POINTER(C.c_double), C.POINTER(C.c_double)]
        _lib.wnwo_get_base_slots.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_select_segments.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int), C.c_int, C.c_int, C.POINTER(C.c_int),
                                              C.POINTER(C.c_int), C.POINTER(C.c_int)]
        _lib.wnwo_lag_update.argtypes = [C.POINTER(C.c_int), C.POINTER(C.c_longlong), C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int,
                                         C.c_longlong, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
                                         C.POINTER(C.c_int), C.POINTER(C.c_int)]
        _lib.wnwo_retention_schedule.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_double, C.POINTER(C.c_double)]
        _lib.wnwo_retention_schedule.restype = None
        _lib.wnwo_select_tokens.argtypes = [C.POINTER(C.c_float), C.c_int, C.c_int, C.c_float, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_place_prefill_tokens.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16),
                                                   C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.c_int,
                                                   C.POINTER(C.c_float), C.c_int, C.c_int]
        _lib.wnwo_get_token_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_double)]
        _lib.wnwo_get_fixed_tokens.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_set_fixed_tokens.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int]
        _lib.wnwo_topk.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int), C.c_int, C.c_int, C.POINTER(C.c_int)]
        _lib.wnwo_table_update.argtypes = [C.POINTER(C.c_int), C.POINTER(C.c_longlong), C.c_int, C.POINTER(C.c_int), C.c_int,
                                           C.c_longlong, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
                                           C.POINTER(C.c_int)]
    return _lib


class OracleError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        raise OracleError(f"{what}: oracle status {rc}")


def topk(score_sum: np.ndarray, lens: np.ndarray, k: int) -> np.ndarray:
    """Rank chunks by (float32 mean desc, index asc); the first min(k, C) of them."""
    s = np.ascontiguousarray(score_sum, dtype=np.float32)
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    out = np.full(max(k, 1), -1, dtype=np.int32)
    n = lib().wnwo_topk(_p(s, C.c_float), _p(ln, C.c_int), len(s), k, _p(out, C.c_int))
    return out[:n].copy()


def table_update(slot_chunk: np.ndarray, stamp: np.ndarray, sel: Sequence[int], step: int, topk_cfg: int):
    """Apply one chunk-swap update in place.  Returns (plan [(chunk, slot, evicted)], n_hits)."""
    assert slot_chunk.dtype == np.int32 and stamp.dtype == np.int64
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    k = len(sel)
    pc = np.zeros(max(k, 1), np.int32); ps = np.zeros(max(k, 1), np.int32); ev = np.zeros(max(k, 1), np.int32)
    hits = C.c_int(0)
    n = lib().wnwo_table_update(_p(slot_chunk, C.c_int), _p(stamp, C.c_longlong), len(slot_chunk), _p(sel, C.c_int), k,
                                step, topk_cfg, _p(pc, C.c_int), _p(ps, C.c_int), _p(ev, C.c_int), C.byref(hits))
    if n < 0:
        raise OracleError("table_update: no victim (S < k?)")
    return [(int(pc[i]), int(ps[i]), int(ev[i])) for i in range(n)], hits.value


def retention_schedule(s_tilde, lam: float) -> np.ndarray:
    """Eq. 1: retention_i = min(s_tilde_i * lambda, 1)."""
    st = np.ascontiguousarray(s_tilde, np.float64)
    out = np.zeros(len(st), np.float64)
    lib().wnwo_retention_schedule(_p(st, C.c_double), len(st), float(lam), _p(out, C.c_double))
    return out


def select_tokens(key: np.ndarray, seg: int, retention: float, variant: int = 0) -> np.ndarray:
    """Kept positions of a fixed head ("Prefill Compression"): per-segment top floor(retention * n_s) (variant 0) or the
    same total taken from the whole head (variant 1, the ablation's global top-k)."""
    kf = np.ascontiguousarray(key, np.float32)
    out = np.zeros(max(len(kf), 1), np.int32)
    n = lib().wnwo_select_tokens(_p(kf, C.c_float), len(kf), int(seg), float(retention), int(variant), _p(out, C.c_int))
    _check(-min(n, 0), "select_tokens")
    return out[:n].copy()


def select_segments(seg_sum: np.ndarray, lens: np.ndarray, k: int):
    """Overlapping chunks (chunk j = segments j, j+1): the k best chunks in rank order and their segments, in that order
    without repeats.  Returns (chunks, segments)."""
    s = np.ascontiguousarray(seg_sum, dtype=np.float32)
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    ch = np.full(max(k, 1), -1, dtype=np.int32)
    sg = np.full(max(2 * k, 1), -1, dtype=np.int32)
    n_sel = C.c_int(0)
    n = lib().wnwo_select_segments(_p(s, C.c_float), _p(ln, C.c_int), len(s), k, _p(ch, C.c_int), C.byref(n_sel), _p(sg, C.c_int))
    if n < 0:
        raise OracleError("select_segments failed")
    return ch[:n_sel.value].copy(), sg[:n].copy()


def lag_update(slot_seg: np.ndarray, stamp: np.ndarray, s_base: int, segs: Sequence[int], step: int, delta: int):
    """Apply one segment swap with permanent base slots [0, s_base) and lag-delta release, in place.
    Returns (plan [(segment, slot)], released segments, n_hits)."""
    assert slot_seg.dtype == np.int32 and stamp.dtype == np.int64
    segs = np.ascontiguousarray(segs, dtype=np.int32)
    n = len(segs)
    pg = np.zeros(max(n, 1), np.int32); pj = np.zeros(max(n, 1), np.int32); rel = np.zeros(max(len(slot_seg), 1), np.int32)
    n_rel, hits = C.c_int(0), C.c_int(0)
    m = lib().wnwo_lag_update(_p(slot_seg, C.c_int), _p(stamp, C.c_longlong), s_base, len(slot_seg), _p(segs, C.c_int), n, step,
                              delta, _p(pg, C.c_int), _p(pj, C.c_int), _p(rel, C.c_int), C.byref(n_rel), C.byref(hits))
    if m < 0:
        raise OracleError("lag_update: no free dynamic slot")
    return [(int(pg[i]), int(pj[i])) for i in range(m)], [int(x) for x in rel[:n_rel.value]], hits.value


class Oracle:
    """The stateful decode-step oracle.  Arrays in/out are numpy; bf16 values travel as uint16 bit patterns."""

    def __init__(self, n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_audio_tokens, max_text_tokens,
                 chunk_tokens, topk, budget, roles, softmax_scale=0.0, score_scope=0, residency=0, evict_lag=3,
                 global_anchor_layers=None):
        self.L, self.Hq, self.Hkv, self.d = n_layers, n_q_heads, n_kv_heads, head_dim
        self.topk_cfg = topk
        roles = np.ascontiguousarray(roles, dtype=np.uint8).reshape(-1)
        assert roles.size == n_layers * n_kv_heads
        h = C.c_void_p()
        # budget is a float32 field in the library's config; mirror that rounding here
        # global_anchor_layers [n_layers]: this oracle holds one shard of the KV heads (see wnwo_create_shard)
        ga = None if global_anchor_layers is None else np.ascontiguousarray(global_anchor_layers, dtype=np.uint8)
        _check(lib().wnwo_create_shard(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_audio_tokens, max_text_tokens,
                                       chunk_tokens, topk, float(np.float32(budget)), float(softmax_scale),
                                       _p(roles, C.c_uint8), score_scope, residency, evict_lag, _p(ga, C.c_uint8), C.byref(h)),
               "create")
        self.residency_mode, self.evict_lag = residency, evict_lag
        self.score_scope = score_scope
        self._h = h
        self._n_active = 0

    def close(self):
        if self._h:
            lib().wnwo_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def base_slots(self, seq: int) -> int:
        """Slots of the tidal tables that were filled at prefill (all of them under the hard budget)."""
        v = C.c_int(0)
        _check(lib().wnwo_get_base_slots(self._h, seq, C.byref(v)), "get_base_slots")
        return v.value

    def score_source(self, layer: int) -> int:
        return lib().wnwo_score_source(self._h, layer)

    def place_prefill(self, seq, layer, k_bits, v_bits, audio_begin, audio_end, q_last_bits):
        k_bits, v_bits = _u16(k_bits), _u16(v_bits)
        n = k_bits.shape[0]
        assert k_bits.shape == v_bits.shape == (n, self.Hkv, self.d)
        q = None if q_last_bits is None else _u16(q_last_bits)   # [Hq, d], or [n_q, Hq, d]: all the text queries
        n_q = 1 if q is None or q.ndim == 2 else q.shape[0]
        _check(lib().wnwo_place_prefill_multi(self._h, seq, layer, _p(k_bits, C.c_uint16), _p(v_bits, C.c_uint16), n, audio_begin,
                                              audio_end, _p(q, C.c_uint16), n_q), "place_prefill")

    def place_prefill_tokens(self, seq, layer, k_bits, v_bits, audio_begin, audio_end, q_text_bits, retention, seg, variant=0):
        k = _u16(k_bits); v = _u16(v_bits); q = _u16(q_text_bits)
        n_q = q.size // (self.Hq * self.d)
        r = np.ascontiguousarray(retention, np.float32)
        assert len(r) == self.Hkv
        _check(lib().wnwo_place_prefill_tokens(self._h, seq, layer, _p(k, C.c_uint16), _p(v, C.c_uint16), k.shape[0],
                                               audio_begin, audio_end, _p(q, C.c_uint16), n_q, _p(r, C.c_float), int(seg),
                                               int(variant)), "place_prefill_tokens")

    def token_scores(self, seq, layer, kv_head) -> np.ndarray:
        out = np.zeros(max(self.dims(seq)[0], 1), np.float64)
        _check(lib().wnwo_get_token_scores(self._h, seq, layer, kv_head, _p(out, C.c_double)), "token_scores")
        return out[:self.dims(seq)[0]]

    def fixed_tokens(self, seq, layer, kv_head):
        out = np.zeros(max(self.dims(seq)[0], 1), np.int32)
        n = lib().wnwo_get_fixed_tokens(self._h, seq, layer, kv_head, _p(out, C.c_int))
        return None if n < 0 else out[:n].copy()

    def set_fixed_tokens(self, seq, layer, kv_head, pos):
        a = np.ascontiguousarray(pos, np.int32)
        _check(lib().wnwo_set_fixed_tokens(self._h, seq, layer, kv_head, _p(a, C.c_int), len(a)), "set_fixed_tokens")

    def append_audio(self, seq, k_bits, v_bits):
        """The clip of `seq` grows by n audio positions: k_bits, v_bits [n_layers, n, n_kv_heads, head_dim] (every layer)."""
        k, v = _u16(k_bits), _u16(v_bits)
        assert k.shape == v.shape and k.shape[0] == self.L and k.shape[2:] == (self.Hkv, self.d), k.shape
        _check(lib().wnwo_append_audio(self._h, seq, _p(k, C.c_uint16), _p(v, C.c_uint16), k.shape[1]), "append_audio")

    def step_begin(self, active: Sequence[int]):
        a = np.ascontiguousarray(active, dtype=np.int32)
        _check(lib().wnwo_step_begin(self._h, _p(a, C.c_int), len(a)), "step_begin")
        self._n_active = len(a)

    def decode_layer(self, layer, q_bits, k_new_bits=None, v_new_bits=None) -> np.ndarray:
        q = _u16(q_bits)
        assert q.shape == (self._n_active, self.Hq, self.d), q.shape
        kn = None if k_new_bits is None else _u16(k_new_bits)
        vn = None if v_new_bits is None else _u16(v_new_bits)
        out = np.zeros((self._n_active, self.Hq, self.d), dtype=np.float64)
        _check(lib().wnwo_decode_layer(self._h, layer, _p(q, C.c_uint16), _p(kn, C.c_uint16), _p(vn, C.c_uint16),
                                       _p(out, C.c_double)), "decode_layer")
        return out

    def step_end(self):
        _check(lib().wnwo_step_end(self._h), "step_end")

    def dims(self, seq) -> Tuple[int, int, int, int]:
        v = [C.c_int() for _ in range(4)]
        _check(lib().wnwo_get_dims(self._h, seq, *[C.byref(x) for x in v]), "get_dims")
        return tuple(x.value for x in v)  # T_a, T_t, C, S

    def chunk_scores(self, seq, layer) -> np.ndarray:
        out = np.zeros(self.dims(seq)[2], np.float64)
        lib().wnwo_get_chunk_scores(self._h, seq, layer, _p(out, C.c_double))
        return out

    def set_chunk_scores(self, seq, layer, scores):
        sc = np.ascontiguousarray(scores, np.float64)
        assert len(sc) == self.dims(seq)[2]
        _check(lib().wnwo_set_chunk_scores(self._h, seq, layer, _p(sc, C.c_double)), "set_chunk_scores")

    def prefill_scores(self, seq, layer, kv_head) -> np.ndarray:
        out = np.zeros(self.dims(seq)[2], np.float64)
        lib().wnwo_get_prefill_scores(self._h, seq, layer, kv_head, _p(out, C.c_double))
        return out

    def selected(self, seq, layer) -> np.ndarray:
        out = np.full(self.topk_cfg, -1, np.int32)
        n = lib().wnwo_get_selected(self._h, seq, layer, _p(out, C.c_int))
        return out[:n].copy()

    def residency(self, seq, layer) -> Tuple[np.ndarray, np.ndarray]:
        S = self.dims(seq)[3]
        sc = np.zeros(S, np.int32); st = np.zeros(S, np.int64)
        lib().wnwo_get_residency(self._h, seq, layer, _p(sc, C.c_int), _p(st, C.c_longlong))
        return sc, st

    def set_residency(self, seq, layer, slot_chunk, stamp):
        sc = np.ascontiguousarray(slot_chunk, np.int32); st = np.ascontiguousarray(stamp, np.int64)
        assert len(sc) == len(st) == self.dims(seq)[3]
        lib().wnwo_set_residency(self._h, seq, layer, _p(sc, C.c_int), _p(st, C.c_longlong))

    def fixed_set(self, seq, layer, kv_head) -> np.ndarray:
        out = np.full(max(self.dims(seq)[3], 1), -1, np.int32)
        n = lib().wnwo_get_fixed_set(self._h, seq, layer, kv_head, _p(out, C.c_int))
        return out[:n].copy()

    def set_fixed_set(self, seq, layer, kv_head, chunks):
        c = np.ascontiguousarray(chunks, np.int32)
        _check(lib().wnwo_set_fixed_set(self._h, seq, layer, kv_head, _p(c, C.c_int), len(c)), "set_fixed_set")

    def stats(self, seq) -> dict:
        v = [C.c_longlong() for _ in range(3)]
        lib().wnwo_get_stats(self._h, seq, *[C.byref(x) for x in v])
        return {"hits": v[0].value, "misses": v[1].value, "evictions": v[2].value}

    def attention_row(self, seq, layer, q_head, q_bits) -> Tuple[np.ndarray, np.ndarray]:
        T_a, T_t, _, _ = self.dims(seq)
        q = _u16(q_bits).reshape(self.d)
        p = np.zeros(T_t + T_a, np.float64); out = np.zeros(self.d, np.float64)
        _check(lib().wnwo_attention_row(self._h, seq, layer, q_head, _p(q, C.c_uint16), _p(p, C.c_double),
                                        _p(out, C.c_double)), "attention_row")
        return p, out
