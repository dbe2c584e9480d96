"""Randomised small configurations: roles, group size, head_dim, chunk, budget, batch, ragged lengths, routing, eager and
graph replay mixed.  Every case runs the full lock-step parity check against the oracle (needs a B200)."""
import numpy as np
import pytest

from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, tiny_custom

pytestmark = pytest.mark.gpu


def _draw(seed):
    rs = np.random.RandomState(1000 + seed)
    n_layers = int(rs.randint(1, 6))
    hkv = int(rs.choice([1, 2, 4, 8]))
    g = int(rs.choice([1, 2, 4, 8, 16]))
    while hkv * g > 128:
        g //= 2
    d = int(rs.choice([64, 128]))
    chunk = int(rs.choice([16, 32, 64, 25, 50, 40, 9]))
    batch = int(rs.randint(1, 4))
    lens = [int(rs.randint(0, 12) * chunk + rs.randint(0, chunk)) for _ in range(batch)]
    if sum(lens) == 0:
        lens[0] = chunk * 3 + 5
    roles = rs.choice([ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED], size=(n_layers, hkv), p=[0.25, 0.45, 0.3]).astype(np.uint8)
    if not (roles == ROLE_ANCHOR).any():
        roles[rs.randint(n_layers), rs.randint(hkv)] = ROLE_ANCHOR
    return tiny_custom(n_layers=n_layers, n_q_heads=hkv * g, n_kv_heads=hkv, head_dim=d, n_text=int(rs.randint(0, 40)),
                       audio_lens=tuple(lens), chunk=chunk, budget=float(rs.choice([0.1, 0.25, 0.5, 1.0])), n_steps=6,
                       roles=roles, topk=int(rs.randint(1, 5)), region=chunk, jump_every=int(rs.choice([0, 2])),
                       name=f"fuzz{seed}"), rs


@pytest.mark.parametrize("seed", range(16))
def test_random_configuration(seed):
    from parity_harness import Lockstep
    w, rs = _draw(seed)
    ls = Lockstep(w, seed=seed)
    try:
        ls.prefill()
        use_graph = bool(seed % 2)
        for t in range(w.n_steps):
            ls.decode_step(t, append=True, graph=use_graph and t not in (0, 3), check_slots=True)
        ls.check_stats()
    finally:
        ls.close()


@pytest.mark.parametrize("seed", range(16))
def test_random_configuration_segment_lag(seed):
    """The same random shapes under SEGMENT_LAG residency with a random eviction lag, score scope and layer ordering."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    w, rs = _draw(seed)
    delta = int(rs.randint(0, 4))
    ls = Lockstep(w, seed=seed, residency=wnw.WNW_RESIDENCY_SEGMENT_LAG, evict_lag=delta, score_scope=int(rs.randint(0, 2)))
    try:
        wnw.wnw_set_layer_dependency(ls.h, int(rs.randint(0, 4)))
        ls.prefill()
        use_graph = bool(seed % 2)
        for t in range(w.n_steps):
            ls.decode_step(t, append=True, graph=use_graph and t not in (0, 3), check_slots=True)
        ls.check_stats()
    finally:
        ls.close()


@pytest.mark.parametrize("seed", range(16))
def test_random_configuration_token_compression(seed):
    """The same random shapes with token-granular prefill compression: fixed heads under every residency (random segment
    size and variant), tidal heads' permanent base under SEGMENT_LAG_TOKEN_BASE; random per-head retention within what a
    compact store holds, random number of text queries, eviction lag, score scope and layer ordering."""
    import paper_2608_22704_b200 as wnw
    from parity_harness import Lockstep
    w, rs = _draw(seed)
    residency = int(rs.choice([0, 1, 2, 2]))
    delta = int(rs.randint(0, 4))
    w.n_prefill_queries = int(rs.randint(1, 4))
    T_max = max(w.audio_lens)
    C = -(-T_max // w.chunk)
    base = min(C, max(1, int(np.floor(float(np.float32(w.budget)) * C + 1e-6))))
    blocks = base + (min(2 * w.topk * (delta + 1), C - base) if residency else 0)
    r_max = min(1.0, 0.95 * blocks * w.chunk / max(T_max, 1))
    ret = (rs.rand(w.n_layers, w.n_kv_heads) * r_max).astype(np.float32)
    ret[rs.rand(w.n_layers, w.n_kv_heads) < 0.1] = 0.0
    seg = w.chunk if residency == 2 else int(rs.choice([w.chunk, 25, 7]))
    variant = int(rs.randint(0, 2))
    ls = Lockstep(w, seed=seed, residency=residency, evict_lag=delta, score_scope=int(rs.randint(0, 2)), token_retention=ret,
                  token_seg=seg, token_variant=variant)
    try:
        wnw.wnw_set_layer_dependency(ls.h, int(rs.randint(0, 4)))
        ls.prefill()
        use_graph = bool(seed % 2)
        for t in range(w.n_steps):
            ls.decode_step(t, append=True, graph=use_graph and t not in (0, 3), check_slots=True)
        ls.check_stats()
    finally:
        ls.close()
