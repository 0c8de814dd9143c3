"""Pins for the oracle's encode, scale and special values.

The oracle finds the nearest value by exhaustive search.  It is pinned here
against (a) the paper's printed Table I values used as an independent grid,
(b) the encoder as Section III-B.2 describes it -- put (exponent + 1) ones at
the top, a terminating zero, then the leading mantissa bits -- written out
with exact rationals and round-half-to-even, (c) idempotence and
monotonicity over every code of every width.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dybit_oracle as orc

FORMATS = [(b, s) for b in range(2, 9) for s in (False, True)]


def _m(bits, signed):
    return bits - 1 if signed else bits


def _nextafter32(x, direction):
    return np.nextafter(np.float32(x), np.float32(direction), dtype=np.float32)


def _table1(golden_dir):
    vals = {}
    with open(os.path.join(golden_dir, "table1_unsigned4.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                p, v = line.split()
                vals[int(p, 2)] = Fraction(v)
    return vals


def _section_encoder(t: Fraction, m: int) -> int:
    """Encoder of Section III-B.2 with exact arithmetic and round-half-to-even.

    t >= 1: exponent e = floor(log2 t); e+1 ones, a zero, then the k = m-2-e
    leading fraction bits of t / 2^e, rounded; a carry out of the fraction
    runs into the unary field, which is what the next binade's first code is.
    t < 1: the m-1 fraction bits of t, rounded.
    """
    vmax = Fraction(2) ** (m - 1)
    if t >= vmax:
        return (1 << m) - 1
    if t < 1:
        scaled = t * 2 ** (m - 1)
        base = 0
    else:
        e = 0
        while Fraction(2) ** (e + 1) <= t:
            e += 1
        k = m - 2 - e
        base = ((1 << (e + 1)) - 1) << (k + 1)
        scaled = (t / Fraction(2) ** e - 1) * 2 ** k
    q = math.floor(scaled)
    rem = scaled - q
    code = base + q
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and code % 2 == 1):
        code += 1
    return code


@pytest.mark.parametrize("bits,signed", FORMATS)
def test_every_code_is_a_fixed_point(bits, signed):
    m = _m(bits, signed)
    tab = orc.decode_table(bits, signed)
    for c in range(1 << bits):
        if signed and c == (1 << m):
            # the redundant "minus zero" pattern is never produced
            assert orc.encode_one(tab[c], 1.0, bits, signed) == 0
            continue
        assert orc.encode_one(tab[c], 1.0, bits, signed) == c
    # decode(encode(x)) is a fixed point of decode∘encode for arbitrary x
    rng = np.random.default_rng(5)
    for x in rng.normal(0, 2 ** (m - 2), 200).astype(np.float32):
        c = orc.encode_one(x, 1.0, bits, signed)
        assert orc.encode_one(orc.decode(bits, signed, c), 1.0, bits, signed) == c


def test_nearest_against_printed_table(golden_dir):
    tab = _table1(golden_dir)
    grid = [Fraction(i, 256) for i in range(0, 10 * 256)]
    for t in grid:
        c = orc.encode_one(float(t), 1.0, 4, False)
        d = abs(t - tab[c])
        best = min(abs(t - v) for v in tab.values())
        assert d == best, (t, c)
        ties = [k for k, v in tab.items() if abs(t - v) == best]
        if len(ties) > 1:
            assert c % 2 == 0 and c in ties


@pytest.mark.parametrize("m", range(1, 9))
def test_matches_the_section_encoder_on_midpoints_and_neighbours(m):
    vals = [Fraction(orc.decode_mag(m, c)) for c in range(1 << m)]
    probes = []
    for a, b in zip(vals, vals[1:]):
        mid = (a + b) / 2
        lo, hi = _nextafter32(float(mid), 0.0), _nextafter32(float(mid), np.inf)
        probes += [a, mid, Fraction(float(lo)), Fraction(float(hi)), (3 * a + b) / 4, (a + 3 * b) / 4]
    probes += [vals[-1], vals[-1] * 3, Fraction(1, 1 << 20), Fraction(0)]
    for t in probes:
        assert float(t) == np.float32(float(t))          # representable: no input rounding
        got = orc.encode_one(float(t), 1.0, m, False)
        assert got == _section_encoder(t, m), (m, t)


@pytest.mark.parametrize("m", range(1, 9))
def test_midpoints_go_to_the_even_code(m):
    vals = [orc.decode_mag(m, c) for c in range(1 << m)]
    for c in range((1 << m) - 1):
        mid = (vals[c] + vals[c + 1]) / 2
        even = c if c % 2 == 0 else c + 1
        assert orc.encode_one(mid, 1.0, m, False) == even
        assert orc.encode_one(_nextafter32(mid, 0.0), 1.0, m, False) == c
        assert orc.encode_one(_nextafter32(mid, np.inf), 1.0, m, False) == c + 1


@pytest.mark.parametrize("bits,signed", FORMATS)
def test_encode_is_monotone_and_random_inputs_match_section_encoder(bits, signed):
    m = _m(bits, signed)
    rng = np.random.default_rng(bits * 2 + signed)
    x = np.sort(np.abs(rng.normal(0, 2 ** (m - 1) / 3, 3000)).astype(np.float32))
    inv = np.float32(0.8125)
    codes = orc.quantize(x, bits, signed, inv)
    assert np.all(np.diff(codes.astype(np.int32)) >= 0)
    for xi, ci in zip(x[::7], codes[::7]):
        t = Fraction(float(np.float32(xi) * inv))
        assert int(ci) == _section_encoder(t, m)
    if signed:
        neg = orc.quantize(-x, bits, signed, inv)
        nz = codes != 0
        assert np.array_equal(neg[nz], codes[nz] | (1 << m))
        assert np.all(neg[~nz] == 0)
    else:
        assert np.all(orc.quantize(-x, bits, signed, inv) == 0)


@pytest.mark.parametrize("bits,signed", FORMATS)
def test_special_values_and_saturation(bits, signed):
    m = _m(bits, signed)
    ones = (1 << m) - 1
    assert orc.encode_one(np.nan, 1.0, bits, signed) == 0
    assert orc.encode_one(np.inf, 1.0, bits, signed) == ones
    assert orc.encode_one(3e38, 1e30, bits, signed) == ones      # product overflows to inf
    assert orc.encode_one(2.0 ** (m - 1) * 1.5, 1.0, bits, signed) == ones
    assert orc.encode_one(3e38, 1.0, bits, signed) == ones            # finite, far beyond double's exact range of distances
    assert orc.encode_one(1e20, 1.0, bits, signed) == ones
    assert orc.encode_one(0.0, 1.0, bits, signed) == 0
    assert orc.encode_one(-0.0, 1.0, bits, signed) == 0
    assert orc.encode_one(-1e-30, 1.0, bits, signed) == 0
    if signed:
        assert orc.encode_one(-np.inf, 1.0, bits, signed) == (1 << m) | ones
    else:
        assert orc.encode_one(-np.inf, 1.0, bits, signed) == 0


@pytest.mark.parametrize("bits,signed", FORMATS)
def test_max_abs_scale(bits, signed):
    m = _m(bits, signed)
    rng = np.random.default_rng(11)
    x = rng.normal(0, 0.02, 4097).astype(np.float32)
    x[100] = np.nan
    x[200] = np.inf
    x[300] = -np.inf
    amax = np.max(np.abs(x[np.isfinite(x)]))
    scale, inv = orc.absmax_scale(x, bits, signed)
    assert scale == np.float32(amax) * np.float32(2.0 ** -(m - 1))
    assert inv == np.float32(2.0 ** (m - 1)) / np.float32(amax)
    # the element that attains the maximum takes the all-ones magnitude
    i = int(np.nanargmax(np.where(np.isfinite(x), np.abs(x), -1)))
    c = orc.encode_one(x[i], inv, bits, signed)
    if signed or x[i] > 0:
        assert c & ((1 << m) - 1) == (1 << m) - 1
    # dequantised maximum is amax again (power-of-two scale: exact)
    assert abs(orc.dequantize(np.array([c], np.uint8), bits, signed, scale)[0]) in (np.float32(amax), 0.0)
    # degenerate tensors
    assert orc.absmax_scale(np.zeros(7, np.float32), bits, signed) == (1.0, 1.0)
    assert orc.absmax_scale(np.zeros(0, np.float32), bits, signed) == (1.0, 1.0)
    assert orc.absmax_scale(np.array([np.nan, np.inf], np.float32), bits, signed) == (1.0, 1.0)
    assert np.all(orc.quantize(np.zeros(7, np.float32), bits, signed, 1.0) == 0)


def test_quantisation_error_is_within_half_a_step():
    # |t - value(code)| <= half the local spacing, for every width
    rng = np.random.default_rng(3)
    for m in range(2, 9):
        vals = np.array([orc.decode_mag(m, c) for c in range(1 << m)])
        t = np.abs(rng.normal(0, 2 ** (m - 1) / 3, 2000)).astype(np.float32)
        t = t[t <= vals[-1]]
        codes = orc.quantize(t, m, False, 1.0).astype(np.int64)
        err = np.abs(t.astype(np.float64) - vals[codes])
        gap_up = np.where(codes < (1 << m) - 1, vals[np.minimum(codes + 1, (1 << m) - 1)] - vals[codes], np.inf)
        gap_dn = np.where(codes > 0, vals[codes] - vals[np.maximum(codes - 1, 0)], np.inf)
        above = t.astype(np.float64) >= vals[codes]
        assert np.all(err <= np.where(above, gap_up, gap_dn) / 2)
