"""Head-sharded serving: the KV heads of every layer are dealt out over ranks, one process per GPU.

Attention is independent per KV head; the one thing that crosses heads is the chunk-score vector of Eq. 2 (anchor
heads' softmax mass per chunk), which ranks every tidal layer's chunks.  So a rank holds a cache over its own heads,
created with the model-wide flags of which layers have an anchor head (score routing follows those) and with the
selection deferred to the end of the step; per step the ranks' partial score sums are added up with ONE all-reduce of
[n_active][n_layers][C_max] floats, handed back, and every rank makes the same selection for its own tidal heads and
recalls over its own host link.  This module is the plumbing: the shard plan and the order of calls of a step.  The
sums themselves are the collective's (NCCL over NVLink on GPUs; gloo in the CPU test).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Sequence

import numpy as np

from . import binding as wnw


@dataclass
class HeadShard:
    rank: int
    world: int
    kv_heads: List[int]              # the model's KV heads this rank holds (ascending)
    q_heads: List[int]               # their query heads, in the order of the rank's own q tensor
    roles: np.ndarray                # uint8 [n_layers, len(kv_heads)]
    global_anchor_layers: np.ndarray  # uint8 [n_layers]: the layer has an anchor head on SOME rank


def shard_plan(roles: np.ndarray, n_q_heads: int, world: int) -> List[HeadShard]:
    """Contiguous blocks of KV heads per rank (a GQA group stays on one rank).  n_kv_heads must divide by world."""
    roles = np.asarray(roles, np.uint8)
    n_layers, n_kv = roles.shape
    if world < 1 or n_kv % world or n_q_heads % n_kv:
        raise ValueError(f"{n_kv} KV heads / {n_q_heads} query heads do not split over {world} ranks")
    per, g = n_kv // world, n_q_heads // n_kv
    flags = (roles == wnw.WNW_ROLE_ANCHOR).any(axis=1).astype(np.uint8)
    plan = []
    for r in range(world):
        kv = list(range(r * per, (r + 1) * per))
        plan.append(HeadShard(r, world, kv, [h * g + j for h in kv for j in range(g)], np.ascontiguousarray(roles[:, kv]), flags.copy()))
    return plan


def create_shard_cache(shard: HeadShard, n_q_heads: int, n_kv_heads: int, head_dim: int, max_batch: int, max_audio_tokens: int,
                       max_text_tokens: int, chunk_tokens: int, budget: float, **kw) -> int:
    """A cache over the rank's own heads: same arguments as wnw_create for the whole model's head counts."""
    g = n_q_heads // n_kv_heads
    return wnw.wnw_create(shard.roles.shape[0], len(shard.kv_heads) * g, len(shard.kv_heads), head_dim, max_batch, max_audio_tokens,
                          max_text_tokens, chunk_tokens, budget, shard.roles, defer_selection=1,
                          global_anchor_layers=shard.global_anchor_layers, **kw)


def sharded_step(cache: int, active: Sequence[int], q, k_new, v_new, out, scores, all_reduce: Callable, stream=None) -> None:
    """One decode step of a shard.  q, k_new, v_new, out: per layer, this rank's heads only (as wnw_decode_layer wants
    them).  scores: a float32 CUDA tensor [len(active), n_layers, C_max] the exchange runs through; all_reduce(scores)
    must add it up over the ranks in place on `stream` (torch.distributed.all_reduce with the nccl backend does)."""
    wnw.wnw_step_begin(cache, list(active))
    for l in range(len(q)):
        wnw.wnw_decode_layer(cache, l, q[l], None if k_new is None else k_new[l], None if v_new is None else v_new[l], out[l],
                             stream=stream)
    wnw.wnw_export_scores(cache, scores, stream=stream)
    all_reduce(scores)
    wnw.wnw_import_scores(cache, scores, stream=stream)
    wnw.wnw_step_end(cache, stream=stream)
