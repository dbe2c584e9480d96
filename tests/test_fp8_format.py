"""The e4m3 storage format of the tidal tier as the tests define it (tests/helpers.py), pinned against things other
than itself: the list of all e4m3 values built from the format's definition, torch's float8_e4m3fn cast (a library
routine), and the properties the scale rule promises."""
import numpy as np
import torch

from helpers import bf16_bits_to_f64, dequantised_tidal_bits, e4m3_round, f32_to_bf16_bits, fp8_scale_exponent
from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL


def _all_e4m3_values():
    vals = []
    for code in range(128):
        E, M = code >> 3, code & 7
        if code == 127:
            continue                                        # the one NaN code of the "fn" variant
        vals.append(M * 2.0 ** -9 if E == 0 else (1 + M / 8) * 2.0 ** (E - 7))
    return np.array(sorted(vals))


def test_grid_points_are_fixed_and_midpoints_go_to_even():
    grid = _all_e4m3_values()
    assert grid[-1] == 448.0 and grid[1] == 2.0 ** -9 and len(grid) == 127
    assert np.array_equal(e4m3_round(grid), grid)
    assert np.array_equal(e4m3_round(-grid[1:]), -grid[1:])
    mid = (grid[:-1] + grid[1:]) / 2
    want = np.where(np.arange(len(mid)) % 2 == 0, grid[:-1], grid[1:])   # codes in order: the even code is the even mantissa
    assert np.array_equal(e4m3_round(mid), want)
    assert np.array_equal(e4m3_round(np.nextafter(mid, np.inf)), grid[1:])
    assert np.array_equal(e4m3_round(np.nextafter(mid, -np.inf)), grid[:-1])
    assert e4m3_round(np.array([1e9]))[0] == 448.0 and e4m3_round(np.array([-500.0]))[0] == -448.0
    assert np.signbit(e4m3_round(np.array([-1e-9]))[0])                  # the sign of a value that rounds to zero is kept


def test_matches_the_library_cast_on_random_values():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.02, 1.0, 30.0, 150.0)])
    x = x[np.abs(x) <= 448.0].astype(np.float32)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(e4m3_round(x.astype(np.float64)), want)


def test_scale_exponent_puts_the_largest_magnitude_in_the_top_binade():
    rng = np.random.default_rng(1)
    for a in np.concatenate([np.abs(rng.standard_normal(2000)) * 10.0 ** rng.uniform(-6, 6, 2000), [448.0, 224.0, 1.75, 1.0, 2.0 ** -20]]):
        a = float(bf16_bits_to_f64(f32_to_bf16_bits(np.array([a], np.float32)))[0])
        if a == 0.0:
            continue
        e = fp8_scale_exponent(a)
        assert 224.0 < a / 2.0 ** e <= 448.0
    assert fp8_scale_exponent(0.0) == 0


def test_dequantised_rows_touch_only_tidal_audio_and_stay_close():
    rng = np.random.default_rng(2)
    T, H, d, ab, ae, chunk = 150, 3, 32, 10, 140, 48          # chunks of 48, 48 and 34 audio rows
    roles = np.array([ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED])
    k = f32_to_bf16_bits((rng.standard_normal((T, H, d)) * rng.uniform(0.1, 8.0, (T, 1, 1))).astype(np.float32))
    v = f32_to_bf16_bits(rng.standard_normal((T, H, d)).astype(np.float32))
    k[20, 1] = 0                                                # a zero row keeps its zeros
    kq, vq = dequantised_tidal_bits(k, v, roles, ab, ae, chunk)
    for src, got in ((k, kq), (v, vq)):
        assert np.array_equal(got[:, [0, 2]], src[:, [0, 2]])   # other roles untouched
        assert np.array_equal(got[:ab], src[:ab]) and np.array_equal(got[ae:], src[ae:])   # text untouched
        a, b = bf16_bits_to_f64(src[ab:ae, 1]), bf16_bits_to_f64(got[ab:ae, 1])
        for c0 in range(0, ae - ab, chunk):
            blk_a, blk_b = a[c0:c0 + chunk], b[c0:c0 + chunk]
            top = np.abs(blk_a).max()
            # three mantissa bits: half a unit in the last place of a normal value is 1/16; values far below the block's
            # largest fall into the subnormal spacing 2^-9 * 2^e <= top * 2^-9 / 224
            assert (np.abs(blk_a - blk_b) <= np.maximum(np.abs(blk_a) / 16, top / 224 * 2.0 ** -10) + 1e-300).all()
            assert np.abs(blk_b).max() <= top * (1 + 1 / 16)
    assert not kq[20, 1].any()
    # idempotent: stored values are on the grid of their own scale
    kq2, vq2 = dequantised_tidal_bits(kq, vq, roles, ab, ae, chunk)
    assert np.array_equal(kq2, kq) and np.array_equal(vq2, vq)


def test_what_the_format_costs_on_the_small_configuration():
    """Two oracles on config 0, one fed the plain prefix and one the values an e4m3 tidal tier stores: decode selections
    are the same (they come from anchor heads, which stay bf16) and outputs move by what three mantissa bits of V allow
    (values of O(1): well under 0.3).  A record of the format's cost, not a parity bar."""
    from helpers import make_oracle
    from workloads import Synth, config0
    from workloads.synth import bf16_bits
    w = config0()
    syn = Synth(w, seed=0)
    plain, stored = make_oracle(w), make_oracle(w)
    try:
        for l in range(w.n_layers):
            p = syn.prefill(0, l)
            kb, vb, qb = bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_last"])
            plain.place_prefill(0, l, kb, vb, p["audio_begin"], p["audio_end"], qb)
            kq, vq = dequantised_tidal_bits(kb, vb, w.roles[l], p["audio_begin"], p["audio_end"], w.chunk)
            stored.place_prefill(0, l, kq, vq, p["audio_begin"], p["audio_end"], qb)
        dec = {l: syn.decode(0, l) for l in range(w.n_layers)}
        worst = 0.0
        for t in range(w.n_steps):
            outs = []
            for o in (plain, stored):
                o.step_begin([0])
                outs.append([o.decode_layer(l, bf16_bits(dec[l]["q"][t])[None], bf16_bits(dec[l]["k_new"][t])[None],
                                            bf16_bits(dec[l]["v_new"][t])[None]) for l in range(w.n_layers)])
                o.step_end()
            for l in range(w.n_layers):
                worst = max(worst, float(np.abs(outs[0][l] - outs[1][l]).max()))
                if (w.roles[l] == ROLE_TIDAL).any():
                    assert plain.selected(0, l).tolist() == stored.selected(0, l).tolist()
        assert 0.0 < worst < 0.3
    finally:
        plain.close(); stored.close()
