"""ctypes binding of include/wnw.h: same names, argument marshalling only.

Device buffers are torch CUDA tensors (torch is used for device memory and streams, nothing else); their
`data_ptr()` goes straight through the C ABI.  Every step of the path runs inside the CUDA library; if the
library is missing this module raises instead of falling back to anything.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

WNW_OK = 0
WNW_ERR_INVALID_ARG, WNW_ERR_STATE, WNW_ERR_OOM_DEVICE, WNW_ERR_OOM_HOST, WNW_ERR_CUDA = 1, 2, 3, 4, 5
WNW_ERR_CAPACITY, WNW_ERR_TIMEOUT, WNW_ERR_UNSUPPORTED, WNW_ERR_DEVICE_CHECK = 6, 7, 8, 9
WNW_ROLE_ANCHOR, WNW_ROLE_TIDAL, WNW_ROLE_FIXED = 0, 1, 2
WNW_MODE_TIERED, WNW_MODE_FULL = 0, 1
WNW_RECALL_SIDE_STREAM, WNW_RECALL_INLINE, WNW_RECALL_SKIP = 0, 1, 2
WNW_SCOPE_PER_LAYER, WNW_SCOPE_GLOBAL = 0, 1
WNW_LAYERS_INDEPENDENT, WNW_LAYERS_CHAINED, WNW_LAYERS_SERIAL, WNW_LAYERS_BATCHED = 0, 1, 2, 3
WNW_RESIDENCY_HARD_BUDGET, WNW_RESIDENCY_SEGMENT_LAG, WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE = 0, 1, 2
WNW_TIDAL_KV_BF16, WNW_TIDAL_KV_FP8_E4M3 = 0, 1


class wnw_config_t(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("max_batch", C.c_int32), ("max_audio_tokens", C.c_int32), ("max_text_tokens", C.c_int32),
                ("chunk_tokens", C.c_int32), ("topk", C.c_int32), ("evict_lag", C.c_int32), ("budget", C.c_float),
                ("softmax_scale", C.c_float), ("roles", C.POINTER(C.c_uint8)), ("device", C.c_int32), ("mode", C.c_int32),
                ("recall_mode", C.c_int32), ("score_scope", C.c_int32), ("residency", C.c_int32), ("defer_selection", C.c_int32),
                ("global_anchor_layers", C.POINTER(C.c_uint8)), ("streaming_audio", C.c_int32), ("tidal_kv_format", C.c_int32)]


class wnw_stats_t(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("steps", "hits", "misses", "evictions", "recall_bytes", "resident_audio_tokens",
                                         "host_audio_tokens", "full_audio_tokens")]


class WnwError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


_lib = None
_vp, _i32 = C.c_void_p, C.c_int32
_SIGNATURES = {
    "wnw_create": [C.POINTER(wnw_config_t), C.POINTER(_vp)],
    "wnw_destroy": [_vp],
    "wnw_place_prefill": [_vp, _i32, _i32, _vp, _vp, _i32, _i32, _i32, _vp, _vp],
    "wnw_place_prefill_multi": [_vp, _i32, _i32, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp],
    "wnw_place_prefill_tokens": [_vp, _i32, _i32, _vp, _vp, _i32, _i32, _i32, _vp, _i32, C.POINTER(C.c_float), _i32, _i32, _vp],
    "wnw_export_scores": [_vp, _vp, _vp],
    "wnw_import_scores": [_vp, _vp, _vp],
    "wnw_export_prefill_tidal": [_vp, _i32, _i32, _vp, _vp],
    "wnw_import_prefill_tidal": [_vp, _i32, _i32, _vp, _vp],
    "wnw_append_audio": [_vp, _i32, _i32, _vp, _vp, _i32, _vp],
    "wnw_retention_schedule": [C.POINTER(C.c_float), _i32, C.c_float, C.POINTER(C.c_float)],
    "wnw_get_token_scores": [_vp, _i32, _i32, _i32, C.POINTER(C.c_float), _i32],
    "wnw_get_fixed_tokens": [_vp, _i32, _i32, _i32, C.POINTER(_i32), _i32, C.POINTER(_i32)],
    "wnw_step_begin": [_vp, C.POINTER(_i32), _i32],
    "wnw_decode_layer": [_vp, _i32, _vp, _vp, _vp, _vp, _vp],
    "wnw_decode_layer_full": [_vp, _i32, _vp, _vp, _vp, _vp, _vp],
    "wnw_step_end": [_vp, _vp],
    "wnw_graph_begin": [_vp, C.POINTER(_i32), _i32, _vp],
    "wnw_graph_end": [_vp, _vp],
    "wnw_graph_launch": [_vp, _vp],
    "wnw_get_chunk_scores": [_vp, _i32, _i32, C.POINTER(C.c_float), C.POINTER(_i32)],
    "wnw_get_prefill_scores": [_vp, _i32, _i32, _i32, C.POINTER(C.c_float), C.POINTER(_i32)],
    "wnw_get_selected": [_vp, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)],
    "wnw_get_residency": [_vp, _i32, _i32, C.POINTER(_i32), C.POINTER(C.c_int64), C.POINTER(_i32)],
    "wnw_get_fixed_set": [_vp, _i32, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)],
    "wnw_get_seq_dims": [_vp, _i32] + [C.POINTER(_i32)] * 4,
    "wnw_get_slot_kv": [_vp, _i32, _i32, _i32, _i32, _i32, _vp],
    "wnw_get_stats": [_vp, C.POINTER(wnw_stats_t)],
    "wnw_set_layer_dependency": [_vp, _i32],
    "wnw_get_launch_counts": [_vp, C.POINTER(C.c_int64)],
    "wnw_debug_advance_step_epoch": [_vp, _i32],
    "wnw_get_base_slots": [_vp, _i32, C.POINTER(_i32)],
    "wnw_set_kernel_timing": [_vp, _i32],
    "wnw_get_kernel_time": [_vp, C.POINTER(C.c_float), C.POINTER(_i32)],
    "wnw_sync": [_vp],
    "wnw_measure_host_link": [_i32, C.c_int64, _i32, C.POINTER(C.c_double), C.POINTER(C.c_double)],
    "wnw_attend_static": [_vp, _i32, _i32, _vp, _vp, _i32, _i32, _i32, C.c_float, _i32, _vp],
    "wnw_attend_static_status": [_i32, _vp, C.POINTER(_i32)],
}


def library_path() -> str:
    return _build.LIB_PATH


def lib():
    """The loaded CUDA library.  Raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2608_22704_b200.build` "
                               "(nvcc, sm_100a). There is no fallback path.")
        _lib = C.CDLL(path)
        for name, args in _SIGNATURES.items():
            fn = getattr(_lib, name)
            fn.argtypes = args
            fn.restype = C.c_int
        _lib.wnw_status_string.argtypes = [C.c_int]
        _lib.wnw_status_string.restype = C.c_char_p
    return _lib


def exported_symbols():
    return list(_SIGNATURES) + ["wnw_status_string"]


def status_string(status: int) -> str:
    return lib().wnw_status_string(status).decode()


def _ck(rc: int, what: str):
    if rc != WNW_OK:
        raise WnwError(rc, what)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    return int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) or None


def wnw_create(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_audio_tokens, max_text_tokens, chunk_tokens,
               budget, roles, topk=3, evict_lag=3, softmax_scale=0.0, device=0, mode=WNW_MODE_TIERED,
               recall_mode=WNW_RECALL_SIDE_STREAM, score_scope=WNW_SCOPE_PER_LAYER, residency=WNW_RESIDENCY_HARD_BUDGET,
               streaming_audio=0, defer_selection=0, global_anchor_layers=None, tidal_kv_format=WNW_TIDAL_KV_BF16) -> int:
    roles = np.ascontiguousarray(roles, dtype=np.uint8).reshape(-1)
    cfg = wnw_config_t(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_audio_tokens, max_text_tokens,
                       chunk_tokens, topk, evict_lag, budget, softmax_scale,
                       roles.ctypes.data_as(C.POINTER(C.c_uint8)), device, mode, recall_mode, score_scope, residency,
                       int(defer_selection), None, int(streaming_audio), int(tidal_kv_format))
    if global_anchor_layers is not None:
        ga = np.ascontiguousarray(global_anchor_layers, dtype=np.uint8).reshape(-1)
        if ga.size != n_layers:
            raise WnwError(WNW_ERR_INVALID_ARG, "wnw_create (global_anchor_layers size)")
        cfg.global_anchor_layers = ga.ctypes.data_as(C.POINTER(C.c_uint8))
    if roles.size != n_layers * n_kv_heads:
        raise WnwError(WNW_ERR_INVALID_ARG, "wnw_create (roles size)")
    h = _vp()
    _ck(lib().wnw_create(C.byref(cfg), C.byref(h)), "wnw_create")
    return h.value


def wnw_destroy(cache: int):
    _ck(lib().wnw_destroy(cache), "wnw_destroy")


def wnw_place_prefill(cache, seq, layer, k, v, audio_begin, audio_end, q_last=None, stream=None):
    """q_last: [n_q_heads, head_dim] (the last prefix query) or [n_queries, n_q_heads, head_dim] (all text queries)."""
    if q_last is not None and q_last.dim() == 3:
        return wnw_place_prefill_multi(cache, seq, layer, k, v, audio_begin, audio_end, q_last, stream)
    _ck(lib().wnw_place_prefill(cache, seq, layer, _ptr(k), _ptr(v), k.shape[0], audio_begin, audio_end, _ptr(q_last),
                                _stream(stream)), "wnw_place_prefill")


def wnw_export_scores(cache, scores, stream=None):
    """scores: float32 CUDA tensor [n_active, n_layers, C_max]."""
    _ck(lib().wnw_export_scores(cache, _ptr(scores), _stream(stream)), "wnw_export_scores")


def wnw_import_scores(cache, scores, stream=None):
    _ck(lib().wnw_import_scores(cache, _ptr(scores), _stream(stream)), "wnw_import_scores")


def wnw_export_prefill_tidal(cache, seq, layer, sums, stream=None):
    """sums: float32 CUDA tensor [C_max]."""
    _ck(lib().wnw_export_prefill_tidal(cache, seq, layer, _ptr(sums), _stream(stream)), "wnw_export_prefill_tidal")


def wnw_import_prefill_tidal(cache, seq, layer, sums, stream=None):
    _ck(lib().wnw_import_prefill_tidal(cache, seq, layer, _ptr(sums), _stream(stream)), "wnw_import_prefill_tidal")


def wnw_append_audio(cache, seq, layer, k, v, stream=None):
    """k, v: [n_tokens, n_kv_heads, head_dim] bf16 CUDA tensors, the new audio positions of one layer."""
    _ck(lib().wnw_append_audio(cache, seq, layer, _ptr(k), _ptr(v), k.shape[0], _stream(stream)), "wnw_append_audio")


def wnw_place_prefill_multi(cache, seq, layer, k, v, audio_begin, audio_end, q_text, stream=None):
    _ck(lib().wnw_place_prefill_multi(cache, seq, layer, _ptr(k), _ptr(v), k.shape[0], audio_begin, audio_end, _ptr(q_text),
                                      q_text.shape[0], _stream(stream)), "wnw_place_prefill_multi")


def wnw_place_prefill_tokens(cache, seq, layer, k, v, audio_begin, audio_end, q_text, retention, segment_tokens, variant=0,
                             stream=None):
    r = np.ascontiguousarray(retention, np.float32)
    _ck(lib().wnw_place_prefill_tokens(cache, seq, layer, _ptr(k), _ptr(v), k.shape[0], audio_begin, audio_end, _ptr(q_text),
                                       q_text.shape[0] if q_text.dim() == 3 else 1, r.ctypes.data_as(C.POINTER(C.c_float)),
                                       segment_tokens, variant, _stream(stream)), "wnw_place_prefill_tokens")


def wnw_retention_schedule(s_tilde, lam: float) -> np.ndarray:
    s = np.ascontiguousarray(s_tilde, np.float32)
    out = np.zeros(len(s), np.float32)
    _ck(lib().wnw_retention_schedule(s.ctypes.data_as(C.POINTER(C.c_float)), len(s), float(lam),
                                     out.ctypes.data_as(C.POINTER(C.c_float))), "wnw_retention_schedule")
    return out


def wnw_step_begin(cache, active: Sequence[int]):
    a = (C.c_int32 * len(active))(*active)
    _ck(lib().wnw_step_begin(cache, a, len(active)), "wnw_step_begin")


def wnw_decode_layer(cache, layer, q, k_new, v_new, out, stream=None):
    _ck(lib().wnw_decode_layer(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)), "wnw_decode_layer")


def wnw_decode_layer_full(cache, layer, q, k_new, v_new, out, stream=None):
    _ck(lib().wnw_decode_layer_full(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream(stream)),
        "wnw_decode_layer_full")


def wnw_step_end(cache, stream=None):
    _ck(lib().wnw_step_end(cache, _stream(stream)), "wnw_step_end")


def wnw_graph_begin(cache, active: Sequence[int], stream=None):
    a = (C.c_int32 * len(active))(*active)
    _ck(lib().wnw_graph_begin(cache, a, len(active), _stream(stream)), "wnw_graph_begin")


def wnw_graph_end(cache, stream=None):
    _ck(lib().wnw_graph_end(cache, _stream(stream)), "wnw_graph_end")


def wnw_graph_launch(cache, stream=None):
    _ck(lib().wnw_graph_launch(cache, _stream(stream)), "wnw_graph_launch")


def wnw_sync(cache):
    _ck(lib().wnw_sync(cache), "wnw_sync")


def wnw_get_seq_dims(cache, seq):
    v = [_i32() for _ in range(4)]
    _ck(lib().wnw_get_seq_dims(cache, seq, *[C.byref(x) for x in v]), "wnw_get_seq_dims")
    return tuple(x.value for x in v)  # T_a, T_t, C, S


def wnw_get_base_slots(cache, seq) -> int:
    v = _i32()
    _ck(lib().wnw_get_base_slots(cache, seq, C.byref(v)), "wnw_get_base_slots")
    return v.value


def wnw_get_chunk_scores(cache, seq, layer) -> np.ndarray:
    n_c = wnw_get_seq_dims(cache, seq)[2]
    out = np.zeros(max(n_c, 1), np.float32)
    n = _i32()
    _ck(lib().wnw_get_chunk_scores(cache, seq, layer, out.ctypes.data_as(C.POINTER(C.c_float)), C.byref(n)), "wnw_get_chunk_scores")
    return out[:n.value].copy()


def wnw_get_prefill_scores(cache, seq, layer, kv_head) -> np.ndarray:
    n_c = wnw_get_seq_dims(cache, seq)[2]
    out = np.zeros(max(n_c, 1), np.float32)
    n = _i32()
    _ck(lib().wnw_get_prefill_scores(cache, seq, layer, kv_head, out.ctypes.data_as(C.POINTER(C.c_float)), C.byref(n)),
        "wnw_get_prefill_scores")
    return out[:n.value].copy()


def wnw_get_selected(cache, seq, layer) -> np.ndarray:
    out = np.full(8, -1, np.int32)
    n = _i32()
    _ck(lib().wnw_get_selected(cache, seq, layer, out.ctypes.data_as(C.POINTER(_i32)), C.byref(n)), "wnw_get_selected")
    return out[:n.value].copy()


def wnw_get_residency(cache, seq, layer):
    S = wnw_get_seq_dims(cache, seq)[3]
    sc = np.full(max(S, 1), -1, np.int32)
    st = np.zeros(max(S, 1), np.int64)
    n = _i32()
    _ck(lib().wnw_get_residency(cache, seq, layer, sc.ctypes.data_as(C.POINTER(_i32)), st.ctypes.data_as(C.POINTER(C.c_int64)),
                                C.byref(n)), "wnw_get_residency")
    return sc[:n.value].copy(), st[:n.value].copy()


def wnw_get_fixed_set(cache, seq, layer, kv_head) -> np.ndarray:
    S = wnw_get_seq_dims(cache, seq)[3]
    out = np.full(max(S, 1), -1, np.int32)
    n = _i32()
    _ck(lib().wnw_get_fixed_set(cache, seq, layer, kv_head, out.ctypes.data_as(C.POINTER(_i32)), C.byref(n)), "wnw_get_fixed_set")
    return out[:n.value].copy()


def wnw_get_token_scores(cache, seq, layer, kv_head) -> np.ndarray:
    T_a = wnw_get_seq_dims(cache, seq)[0]
    out = np.zeros(max(T_a, 1), np.float32)
    _ck(lib().wnw_get_token_scores(cache, seq, layer, kv_head, out.ctypes.data_as(C.POINTER(C.c_float)), len(out)),
        "wnw_get_token_scores")
    return out[:T_a].copy()


def wnw_get_fixed_tokens(cache, seq, layer, kv_head) -> np.ndarray:
    T_a = wnw_get_seq_dims(cache, seq)[0]
    out = np.full(max(T_a, 1), -1, np.int32)
    n = _i32()
    _ck(lib().wnw_get_fixed_tokens(cache, seq, layer, kv_head, out.ctypes.data_as(C.POINTER(_i32)), len(out), C.byref(n)),
        "wnw_get_fixed_tokens")
    return out[:n.value].copy()


def wnw_get_slot_kv(cache, seq, layer, kv_head, slot, which, chunk_tokens, head_dim) -> np.ndarray:
    out = np.zeros((chunk_tokens, head_dim), np.uint16)
    _ck(lib().wnw_get_slot_kv(cache, seq, layer, kv_head, slot, which, out.ctypes.data_as(_vp)), "wnw_get_slot_kv")
    return out


def wnw_get_stats(cache) -> dict:
    s = wnw_stats_t()
    _ck(lib().wnw_get_stats(cache, C.byref(s)), "wnw_get_stats")
    return {n: getattr(s, n) for n, _ in wnw_stats_t._fields_}


def wnw_debug_advance_step_epoch(cache, delta: int):
    _ck(lib().wnw_debug_advance_step_epoch(cache, int(delta)), "wnw_debug_advance_step_epoch")


def wnw_get_launch_counts(cache):
    """(attention, selection, recall, step-end) kernels launched so far, replayed steps included."""
    arr = (C.c_int64 * 4)()
    _ck(lib().wnw_get_launch_counts(cache, arr), "wnw_get_launch_counts")
    return tuple(int(x) for x in arr)


def wnw_set_layer_dependency(cache, mode: int):
    _ck(lib().wnw_set_layer_dependency(cache, int(mode)), "wnw_set_layer_dependency")


def wnw_set_kernel_timing(cache, enable: bool):
    _ck(lib().wnw_set_kernel_timing(cache, int(enable)), "wnw_set_kernel_timing")


def wnw_get_kernel_time(cache):
    ms, n = C.c_float(), _i32()
    _ck(lib().wnw_get_kernel_time(cache, C.byref(ms), C.byref(n)), "wnw_get_kernel_time")
    return ms.value, n.value


def wnw_measure_host_link(device=0, nbytes=256 << 20, reps=5):
    a, b = C.c_double(), C.c_double()
    _ck(lib().wnw_measure_host_link(device, nbytes, reps, C.byref(a), C.byref(b)), "wnw_measure_host_link")
    return a.value, b.value


def wnw_attend_static(kv, n_tokens, q, out, softmax_scale=0.0, stream=None):
    """Full attention of one query token over kv [n_kv_heads, 2, padded_tokens, head_dim] (bf16 CUDA tensor) with no
    allocation inside the library; q, out: [n_q_heads, head_dim] bf16 CUDA tensors."""
    n_kv, two, padded, d = kv.shape
    assert two == 2
    _ck(lib().wnw_attend_static(_ptr(kv), n_tokens, padded, _ptr(q), _ptr(out), q.shape[0], n_kv, d, softmax_scale,
                                kv.device.index or 0, _stream(stream)), "wnw_attend_static")


def wnw_attend_static_status(device: int = 0, stream=None) -> bool:
    """Waits for the stream's queued work; True if a bounded device-side wait of wnw_attend_static ran out since the
    last query (the output of that call is then incomplete).  Clears the flag."""
    v = _i32(0)
    _ck(lib().wnw_attend_static_status(device, _stream(stream), C.byref(v)), "wnw_attend_static_status")
    return bool(v.value)
