"""Pins of the 8-bit cache oracle (oracle/fp8_cache.py) against what the E4M3 format's definition and the
mathematics fix: known codes, the whole code table, nearest-value brute force, tie and saturation cases, and the
reduction of the attention to the plain oracle when nothing is lost in quantisation."""
import numpy as np
import pytest

from oracle import dl_oracle as orc
from oracle import fp8_cache as f8


def test_known_codes_of_the_format():
    # 1-4-3 with bias 7: 0x38 = 0 0111 000 = 1.0; 0x40 = 2.0; 0x3C = 1.5; 0x08 = smallest normal 2^-6;
    # 0x01 = smallest subnormal 2^-9; 0x07 = 7 * 2^-9; 0x7E = 0 1111 110 = 1.75 * 2^8 = 448 (largest); 0x7F = NaN
    vals = {0x00: 0.0, 0x38: 1.0, 0x40: 2.0, 0x3C: 1.5, 0x08: 2.0 ** -6, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9,
            0x7E: 448.0, 0xB8: -1.0, 0xFE: -448.0, 0x30: 0.5, 0x39: 1.125}
    for code, v in vals.items():
        assert f8.e4m3_decode(np.uint8(code)) == v, hex(code)
    assert np.isnan(f8.e4m3_decode(np.uint8(0x7F))) and np.isnan(f8.e4m3_decode(np.uint8(0xFF)))
    assert np.signbit(f8.e4m3_decode(np.uint8(0x80))) and f8.e4m3_decode(np.uint8(0x80)) == 0.0


def test_table_is_monotone_and_round_trips():
    codes = np.arange(0x7F, dtype=np.uint8)
    mags = f8.e4m3_decode(codes)
    assert np.all(np.diff(mags) > 0)
    # spacing: 2^-9 below 2^-6, then 8 steps per binade
    assert np.allclose(np.diff(mags[:9]), 2.0 ** -9)
    assert np.array_equal(f8.e4m3_encode(mags.astype(np.float32)), codes)
    assert np.array_equal(f8.e4m3_encode((-mags).astype(np.float32)), codes | 0x80)


def test_encode_is_the_nearest_value_by_brute_force():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 60, 2000), rng.uniform(-2 ** -5, 2 ** -5, 2000),
                        rng.uniform(-500, 500, 1000)]).astype(np.float32)
    codes = np.arange(256, dtype=np.uint8)
    table = f8.e4m3_decode(codes)
    finite = ~np.isnan(table)
    got = f8.e4m3_encode(x)
    dist = np.abs(table[finite][None, :] - np.clip(x.astype(np.float64), -448, 448)[:, None])
    best = dist.min(axis=1)
    assert np.array_equal(np.abs(f8.e4m3_decode(got) - np.clip(x.astype(np.float64), -448, 448)), best)
    assert np.array_equal(np.signbit(f8.e4m3_decode(got)), np.signbit(x))


def test_ties_go_to_the_even_code_and_large_values_saturate():
    enc = lambda v: int(f8.e4m3_encode(np.float32(v)))
    assert enc(1.0625) == 0x38            # halfway 1.0 (0x38) .. 1.125 (0x39): even code
    assert enc(1.1875) == 0x3A            # halfway 1.125 (0x39) .. 1.25 (0x3A)
    assert enc(np.nextafter(np.float32(1.0625), np.float32(2))) == 0x39
    assert enc(2.0 ** -10) == 0x00        # halfway 0 .. 2^-9
    assert enc(3 * 2.0 ** -10) == 0x02    # halfway 0x01 .. 0x02
    assert enc(-2.0 ** -10) == 0x80       # sign kept on a result of zero
    assert enc(432.0) == 0x7E             # halfway 416 (0x7D) .. 448 (0x7E): even code
    assert enc(448.0) == 0x7E and enc(449.0) == 0x7E and enc(1e30) == 0x7E and enc(-1e30) == 0xFE
    assert enc(np.inf) == 0x7E
    assert enc(np.nan) == 0x7F


def test_quantise_divides_in_float32():
    # x / scale is rounded to float32 before the conversion: a quotient that is a tie only after that rounding
    x, s = np.float32(1.0625) * np.float32(3.0), np.float32(3.0)
    assert int(f8.quantize_rows(x, s)) == int(f8.e4m3_encode(np.float32(x / s)))
    rng = np.random.default_rng(3)
    rows = rng.normal(0, 1, (5, 16)).astype(np.float32)
    sc = np.float32(0.02)
    back = f8.dequantize_rows(f8.quantize_rows(rows, sc), sc)
    # relative step of the format is 2^-3: the nearest value is within 2^-4 relative (or half a subnormal step)
    assert np.all(np.abs(back - rows) <= np.maximum(np.abs(rows) * 2.0 ** -4, 0.5 * 2.0 ** -9 * sc) + 1e-12)


def test_attention_reduces_to_the_plain_oracle_when_rows_are_representable():
    rng = np.random.default_rng(5)
    d, n = 16, 9
    # values that E4M3 holds exactly, scales that are powers of two: nothing is lost
    k = f8.e4m3_decode(rng.integers(0, 0x7E, (n, d)).astype(np.uint8)) * np.where(rng.random((n, d)) < 0.5, -1, 1) / 64
    v = f8.e4m3_decode(rng.integers(0, 0x7E, (n, d)).astype(np.uint8)) / 128
    ks, vs = 2.0 ** -6, 2.0 ** -7
    kc, vc = f8.quantize_rows(k, ks), f8.quantize_rows(v, vs)
    assert np.array_equal(f8.dequantize_rows(kc, ks), k) and np.array_equal(f8.dequantize_rows(vc, vs), v)
    q, kt, vt = rng.normal(0, 1, d), rng.normal(0, 1, d), rng.normal(0, 1, d)
    got = f8.attention_decode_fp8(q, kt, vt, kc, vc, ks, vs, n, 0.25)
    ref = orc.attention_decode_compact(q, kt, vt, k, v, n, 0.25)
    assert np.allclose(got, ref, rtol=0, atol=1e-14)
    # empty cache: the token attends itself only
    assert np.allclose(f8.attention_decode_fp8(q, kt, vt, kc, vc, ks, vs, 0, 0.25), vt)


def test_append_quantises_a_kept_row_and_respects_capacity():
    rng = np.random.default_rng(8)
    d, cap = 8, 3
    kc, vc = np.zeros((cap, d), np.uint8), np.zeros((cap, d), np.uint8)
    kt, vt = rng.normal(0, 1, d).astype(np.float32), rng.normal(0, 1, d).astype(np.float32)
    assert f8.append_row_fp8(kt, vt, 0.05, 0.05, kc, vc, 1, cap, False) == 1 and not kc.any()
    assert f8.append_row_fp8(kt, vt, 0.05, 0.05, kc, vc, 1, cap, True) == 2
    assert np.array_equal(kc[1], f8.quantize_rows(kt, 0.05)) and np.array_equal(vc[1], f8.quantize_rows(vt, 0.05))
    before = kc.copy()
    assert f8.append_row_fp8(kt, vt, 0.05, 0.05, kc, vc, cap, cap, True) == cap and np.array_equal(kc, before)
