"""The allocation-free attention entry point (needs a B200).

wnw_attend_static serves callers that cannot allocate device memory when they need attention (a process whose
device memory all belongs to a pool allocator, a decode thread that cannot take cudaMalloc's device-wide
synchronisation): its scratch is a fixed array inside the library.  The test runs it twice in a row on different
inputs - the array keeps the previous call's contents, so the second call checks that stale scratch does no harm -
and holds each result to two references: textbook softmax attention in float64 (numpy, independent of every kernel
here) and the cache-based entry point wnw_decode_layer_full on a cache holding the same keys and values.  The rows
between n_tokens and padded_tokens are filled with NaN: they are fetched but must never reach the output.  This
file is collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from helpers import bf16_bits_to_f64, dense_attention
from workloads.synth import bf16_bits

pytestmark = pytest.mark.gpu

OUT_TOL = 2e-2   # same bound as the other attention-output parity tests (bf16 outputs of O(1) magnitude)


def _reference_full(wnw, k, v, q, n_q, n_kv, d, device):
    """One decode step of a FULL-mode cache holding k, v [n_tokens, n_kv, d]."""
    n_tokens = k.shape[0]
    roles = np.zeros(n_kv, np.uint8)
    h = wnw.wnw_create(1, n_q, n_kv, d, 1, n_tokens, 16, 16, 1.0, roles, device=device.index or 0, mode=wnw.WNW_MODE_FULL)
    try:
        wnw.wnw_place_prefill(h, 0, 0, k, v, 0, n_tokens)          # every token is audio: no text region
        out = torch.zeros((1, n_q, d), dtype=torch.bfloat16, device=device)
        wnw.wnw_step_begin(h, [0])
        wnw.wnw_decode_layer_full(h, 0, q.unsqueeze(0), None, None, out)
        wnw.wnw_step_end(h)
        wnw.wnw_sync(h)
        return out[0].float().cpu().numpy().astype(np.float64)
    finally:
        wnw.wnw_destroy(h)


def _reference_numpy(k, v, q, n_q, n_kv, d):
    """softmax(q K^T / sqrt d) V per query head in float64 on the bf16 values."""
    K = bf16_bits_to_f64(bf16_bits(k.cpu()))
    V = bf16_bits_to_f64(bf16_bits(v.cpu()))
    Q = bf16_bits_to_f64(bf16_bits(q.cpu()))
    g = n_q // n_kv
    return np.stack([dense_attention(Q[h], K[:, h // g], V[:, h // g], 1.0 / np.sqrt(d))[0] for h in range(n_q)])


@pytest.mark.parametrize("n_q,n_kv,d", [(32, 8, 128), (8, 4, 64), (32, 2, 128), (2, 2, 64)])   # g = 4, 2, 16, 1
def test_attend_static_matches_dense_attention_twice(n_q, n_kv, d):
    import paper_2608_22704_b200 as wnw
    device = torch.device("cuda:0")
    gen = torch.Generator(device="cpu").manual_seed(1234 + n_q)
    for n_tokens in (3000, 517, 9):                    # calls in a row: different sizes, ragged tails, less than one tile
        k = torch.randn(n_tokens, n_kv, d, generator=gen).to(torch.bfloat16).to(device)
        v = torch.randn(n_tokens, n_kv, d, generator=gen).to(torch.bfloat16).to(device)
        q = (torch.randn(n_q, d, generator=gen) * 1.5).to(torch.bfloat16).to(device)
        want = _reference_numpy(k, v, q, n_q, n_kv, d)
        padded = (n_tokens + 15) // 16 * 16 + 16       # a ragged tile and a whole tile of padding
        kv = torch.full((n_kv, 2, padded, d), float("nan"), dtype=torch.bfloat16, device=device)
        kv[:, 0, :n_tokens] = k.permute(1, 0, 2)
        kv[:, 1, :n_tokens] = v.permute(1, 0, 2)
        out = torch.full((n_q, d), float("nan"), dtype=torch.bfloat16, device=device)
        wnw.wnw_attend_static(kv, n_tokens, q, out)
        assert wnw.wnw_attend_static_status(0) is False              # waits for the call; no bounded wait ran out
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= OUT_TOL
        same_path = _reference_full(wnw, k, v, q, n_q, n_kv, d, device)
        assert np.abs(same_path - want).max() <= OUT_TOL
        assert np.abs(got - same_path).max() <= OUT_TOL


def test_attend_static_rejects_sizes_beyond_its_scratch():
    import paper_2608_22704_b200 as wnw
    device = torch.device("cuda:0")
    d = 64
    kv = torch.zeros((128, 2, 16, d), dtype=torch.bfloat16, device=device)       # 128 KV heads > 64
    q = torch.zeros((128, d), dtype=torch.bfloat16, device=device)
    out = torch.zeros_like(q)
    with pytest.raises(wnw.WnwError) as e:
        wnw.wnw_attend_static(kv, 16, q, out)
    assert e.value.status == wnw.WNW_ERR_CAPACITY
