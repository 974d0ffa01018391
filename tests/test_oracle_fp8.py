"""Pins of the e4m3 reference encoder the 8-bit LM-head tests use (oracle/fp8.py): the values the
format's definition fixes, round trips, the tie rule, the error bound, the row-scale rule."""
import numpy as np

from oracle import fp8


def test_code_values_the_format_definition_fixes():
    v = fp8.code_values()
    assert v[0x00] == 0.0 and v[0x01] == 2.0 ** -9 and v[0x07] == 7 * 2.0 ** -9      # subnormals
    assert v[0x08] == 2.0 ** -6                                                      # smallest normal
    assert v[0x38] == 1.0 and v[0x39] == 1.125 and v[0x40] == 2.0
    assert v[0x7E] == 448.0 and len(v) == 127                                        # largest finite; 0x7F is NaN
    assert np.all(np.diff(v) > 0)


def test_every_code_round_trips_and_signs_are_kept():
    codes = np.arange(127, dtype=np.uint8)
    assert np.array_equal(fp8.encode(fp8.decode(codes)), codes)
    neg = codes[1:] | 0x80
    assert np.array_equal(fp8.encode(fp8.decode(neg)), neg)
    assert np.array_equal(fp8.decode(neg), -fp8.decode(codes[1:]))


def test_nearest_code_ties_to_even_and_saturation():
    v = fp8.code_values()
    mid = (v[:-1] + v[1:]) / 2                      # exactly between code c and c + 1
    got = fp8.encode(mid)
    want = np.where(np.arange(126) % 2 == 0, np.arange(126), np.arange(126) + 1)
    assert np.array_equal(got, want.astype(np.uint8))
    assert np.array_equal(fp8.encode(np.nextafter(mid, 0)), np.arange(126).astype(np.uint8))
    assert np.array_equal(fp8.encode(np.nextafter(mid, 1e9)), (np.arange(126) + 1).astype(np.uint8))
    assert fp8.encode(np.array([448.0, 449.0, 1e6, -1e6])).tolist() == [0x7E, 0x7E, 0x7E, 0xFE]


def test_error_bound_and_row_scale_rule():
    rng = np.random.default_rng(0)
    y = rng.standard_normal(200000) * 100
    err = np.abs(fp8.decode(fp8.encode(y)) - y)
    normal = (np.abs(y) >= 2.0 ** -6) & (np.abs(y) <= 448)
    assert np.all(err[normal] <= 2.0 ** -4 * np.abs(y[normal]))
    tiny = rng.uniform(-2.0 ** -6, 2.0 ** -6, 10000)
    assert np.all(np.abs(fp8.decode(fp8.encode(tiny)) - tiny) <= 2.0 ** -10)
    w = (rng.standard_normal((64, 256)) * rng.uniform(1e-3, 10, (64, 1))).astype(np.float32)
    w[7] = 0
    w[9, 0] = 448.0 * 4            # exactly 448 * 2^2: E = 2, not 3
    w[9, 1:] *= 0.01
    s = fp8.row_scales(w)
    amax = np.abs(w).max(axis=1)
    ok = amax > 0
    assert np.all(amax[ok] <= 448 * s[ok]) and np.all(amax[ok] > 224 * s[ok])        # smallest such power of two
    assert s[7] == 1.0 and s[9] == 4.0
    assert np.all(np.log2(s) == np.round(np.log2(s)))
    codes, sc, deq = fp8.quantise_rows(w)
    assert codes.dtype == np.uint8 and np.array_equal(sc, s.astype(np.float32))
    assert np.all(np.abs(deq[ok] - w[ok]) <= 2.0 ** -4 * np.abs(w[ok]) + 2.0 ** -10 * s[ok, None])
    # the dequantised matrix holds 4 significant bits times a power of two: exact in bfloat16
    from paper_2605_18817_b200 import synth
    assert np.array_equal(synth.bf16_round(deq), deq)
