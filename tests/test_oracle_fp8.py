"""Pins for the checker's quantised KV storage (FP8 E4M3 elements, shared power-of-two scale
per head vector).  The E4M3 grid is pinned to hand-written values from the format's definition
and to torch's float8_e4m3fn type (a library routine); rounding to ties, saturation, the scale
rule, scale invariance, idempotence and the error bound are pinned by construction."""
import math

import numpy as np
import pytest
import torch

from oracle import mixattn_oracle as mo


def test_e4m3_grid_hand_values_and_library_decode():
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x0F: 1.875 * 2.0 ** -6,
            0x38: 1.0, 0x3C: 1.5, 0x40: 2.0, 0x77: 240.0, 0x78: 256.0, 0x7E: 448.0, 0xFE: -448.0, 0xB8: -1.0}
    for code, val in hand.items():
        assert mo.e4m3_decode([code])[0] == val, hex(code)
    assert math.isnan(mo.e4m3_decode([0x7F])[0]) and math.isnan(mo.e4m3_decode([0xFF])[0])
    codes = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).double().numpy()
    mine = mo.e4m3_decode(codes)
    fin = ~np.isnan(lib)
    assert fin.sum() == 254 and np.array_equal(np.isnan(mine), ~fin)
    np.testing.assert_array_equal(mine[fin], lib[fin])
    # the grid is strictly increasing over the positive codes
    assert np.all(np.diff(mine[:0x7F]) > 0)


def test_e4m3_encode_round_trip_ties_and_saturation():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    np.testing.assert_array_equal(mo.e4m3_encode(mo.e4m3_decode(codes)), codes)
    pos = mo.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    for c in range(0x7E):
        lo, hi = pos[c], pos[c + 1]
        mid = (lo + hi) / 2                       # exactly representable in float64
        even = c if c % 2 == 0 else c + 1
        assert mo.e4m3_encode([mid])[0] == even, f"tie between codes {c} and {c + 1}"
        assert mo.e4m3_encode([np.nextafter(mid, 0.0)])[0] == c
        assert mo.e4m3_encode([np.nextafter(mid, 1e9)])[0] == c + 1
        assert mo.e4m3_encode([-mid])[0] == (even | 0x80)
    # saturation: everything beyond 448 is 448 (464 would be the tie towards a 480 that does not exist)
    np.testing.assert_array_equal(mo.e4m3_encode([448.0, 449.0, 464.0, 480.0, 511.9, 1e30, -1e30]),
                                  [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE])
    # underflow: at and below half the smallest subnormal the result is (signed) zero
    np.testing.assert_array_equal(mo.e4m3_encode([2.0 ** -10, 2.0 ** -10 * 1.001, 2.0 ** -11, -2.0 ** -11]),
                                  [0x00, 0x01, 0x00, 0x80])


def test_e4m3_encode_matches_library_conversion_in_range():
    rng = np.random.default_rng(1)
    y = np.concatenate([rng.standard_normal(20000) * s for s in (0.01, 1.0, 30.0, 150.0)])
    y = y[np.abs(y) <= 448.0].astype(np.float32)      # (torch converts from fp32; keep inputs fp32-exact)
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(mo.e4m3_encode(y.astype(np.float64)), lib)


def test_shared_exponent_rule_and_scale_invariance():
    # amax = 2^k -> X = k - 8 and the maximum is stored as 256 (code 0x78); amax = 448 * 2^k -> 0x7E
    for k in (-20, -1, 0, 3, 17):
        x = np.zeros((1, 1, 8))
        x[0, 0, 2] = -(2.0 ** k)
        x[0, 0, 5] = 2.0 ** (k - 1)
        codes, X = mo.quantize_kv(x)
        assert X[0, 0] == k - 8 and codes[0, 0, 2] == 0xF8 and codes[0, 0, 5] == 0x70
        x[0, 0, 2] = 448.0 * 2.0 ** k
        codes, X = mo.quantize_kv(x)
        assert X[0, 0] == k and codes[0, 0, 2] == 0x7E
    # a maximum in (448, 512) * 2^X saturates (the one place where the error exceeds half a step)
    codes, X = mo.quantize_kv(np.array([[[500.0, 1.0]]]))
    assert X[0, 0] == 0 and codes[0, 0, 0] == 0x7E and codes[0, 0, 1] == 0x38
    # zero vector
    codes, X = mo.quantize_kv(np.zeros((2, 3, 4)))
    assert (X == -127).all() and (codes == 0).all() and (mo.dequantize_kv(codes, X) == 0).all()
    # multiplying a vector by 2^k moves X by k and leaves the codes alone; each head vector has its own X
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 3, 64)) * np.exp2(rng.integers(-6, 6, size=(5, 3, 1)))
    c0, X0 = mo.quantize_kv(x)
    c1, X1 = mo.quantize_kv(x * 2.0 ** 7)
    np.testing.assert_array_equal(c0, c1)
    np.testing.assert_array_equal(X1, X0 + 7)
    amax = np.abs(x).max(axis=-1)
    np.testing.assert_array_equal(X0, np.floor(np.log2(amax)).astype(int) - 8)
    # K and V rows are independent vectors: changing one row changes nothing in another
    y = x.copy()
    y[0, 0] *= 1000.0
    c2, X2 = mo.quantize_kv(y)
    np.testing.assert_array_equal(c2[1:], c0[1:])
    np.testing.assert_array_equal(c2[0, 1:], c0[0, 1:])


def test_round_trip_error_bound_idempotence_and_bf16_exactness():
    rng = np.random.default_rng(3)
    x = torch.from_numpy(rng.standard_normal((40, 4, 128))).to(torch.bfloat16).double().numpy()
    codes, X = mo.quantize_kv(x)
    r = mo.dequantize_kv(codes, X)
    assert np.array_equal(r, mo.kv_roundtrip(x))
    # half a grid step in the element's binade; the top binade's step is 32 * 2^X <= amax / 8
    scaled = np.abs(x) / np.exp2(X)[..., None]
    e = np.maximum(np.floor(np.log2(np.where(scaled > 0, scaled, 1.0))), -6.0)
    bound = np.where(scaled <= 448.0, np.exp2(e - 4.0), scaled - 448.0) * np.exp2(X)[..., None]
    assert (np.abs(r - x) <= bound).all()
    amax = np.abs(x).max(axis=-1, keepdims=True)
    assert (np.abs(r - x) <= amax / 8.0).all()
    # quantising what was read back changes nothing
    np.testing.assert_array_equal(mo.kv_roundtrip(r), r)
    # the values a quantised cache stands for are bf16 numbers (4 significant bits, power-of-two scale)
    np.testing.assert_array_equal(torch.from_numpy(r).to(torch.bfloat16).double().numpy(), r)
    # and the typical relative error per vector is the E4M3 one (about 2^-5 rms of the elements' size)
    rel = np.linalg.norm(r - x) / np.linalg.norm(x)
    assert 0.01 < rel < 0.04


def test_attention_over_a_quantised_cache_is_attention_over_the_dequantised_values():
    rng = np.random.default_rng(4)
    n, Hq, Hkv, D, W = 50, 4, 2, 16, 9
    q, K, V = rng.standard_normal((Hq, D)), rng.standard_normal((n, Hkv, D)), rng.standard_normal((n, Hkv, D))
    Kq, Vq = mo.kv_roundtrip(K), mo.kv_roundtrip(V)
    for kind in (mo.FULL, mo.SLIDING):
        exact = mo.decode_attention(q, K, V, kind, W)
        quant = mo.decode_attention(q, Kq, Vq, kind, W)
        # dense restatement over the dequantised values (no cache structures)
        lo = 0 if kind == mo.FULL else n - W
        for h in range(Hq):
            g = h // (Hq // Hkv)
            s = (Kq[lo:, g] @ q[h]) / math.sqrt(D)
            w = np.exp(s) / np.exp(s).sum()
            np.testing.assert_allclose(quant[h], w @ Vq[lo:, g], rtol=0, atol=1e-12)
        # quantisation moves the result, by an amount of the size of the E4M3 rounding
        d = np.abs(quant - exact).max()
        assert 0 < d < 0.25
