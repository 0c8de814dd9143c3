"""Pins for the oracle's decode (Eq. 1, Table I, Section III-B.2 worked example).

Nothing here calls the CUDA library.  Expected values come from the paper's
printed table / example (tests/golden) or from facts the format's definition
fixes (monotone codes, dyadic spacing, binade starts at powers of two).
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dybit_oracle as orc

ALL_M = list(range(1, 9))


def _read_golden(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_table_one_printed_values(golden_dir):
    rows = _read_golden(os.path.join(golden_dir, "table1_unsigned4.txt"))
    assert len(rows) == 16
    for pattern, value in rows:
        assert orc.decode(4, False, int(pattern, 2)) == float(value), pattern
        assert orc.decode_mag(4, int(pattern, 2)) == float(value)


def test_worked_decoder_example(golden_dir):
    (pattern, exp_field, man_field), = _read_golden(os.path.join(golden_dir, "decoder_example.txt"))
    code = int(pattern, 2)
    e, man = orc.decode_fields(8, code)
    assert e == int(exp_field, 2)
    assert man == int(man_field, 2)
    # hidden-one mantissa 1.0101000b times 2^exponent
    value = Fraction(int(man_field, 2), 1 << 7) * 2 ** int(exp_field, 2)
    assert value == Fraction(21, 8)
    assert orc.decode(8, False, code) == float(value)


@pytest.mark.parametrize("m", ALL_M)
def test_magnitude_table_structure(m):
    tab = [orc.decode_mag(m, c) for c in range(1 << m)]
    # zero, strictly increasing, hence 2^m distinct values
    assert tab[0] == 0.0
    assert all(b > a for a, b in zip(tab, tab[1:]))
    # largest value and smallest positive value
    assert tab[-1] == 2.0 ** (m - 1)
    if m >= 2:
        assert tab[1] == 2.0 ** -(m - 1)
    # every value is a multiple of 2^-(m-1): integer image, bounded by 4^(m-1)
    ints = [Fraction(v) * 2 ** (m - 1) for v in tab]
    assert all(i.denominator == 1 for i in ints)
    assert max(ints) == 4 ** (m - 1)
    # significant bits never exceed max(m-1, 1)
    for i in ints:
        n = int(i)
        if n:
            while n % 2 == 0:
                n //= 2
            assert n.bit_length() <= max(m - 1, 1)


@pytest.mark.parametrize("m", ALL_M)
def test_sub_unit_codes_are_a_linear_fraction(m):
    for c in range(1 << (m - 1)):               # start bit 0
        assert Fraction(orc.decode_mag(m, c)) == Fraction(c, 1 << (m - 1))


@pytest.mark.parametrize("m", ALL_M)
def test_binades_and_unary_exponent(m):
    # pattern 1^i 0 x_k : value 2^(i-1) * (1 + x / 2^k)
    for i in range(1, m):
        k = m - 1 - i
        head = ((1 << i) - 1) << (k + 1)
        for x in range(1 << k):
            want = Fraction(2) ** (i - 1) * (1 + Fraction(x, 1 << k))
            assert Fraction(orc.decode_mag(m, head | x)) == want
        # binade [2^(i-1), 2^i) holds exactly 2^k codes
        vals = [orc.decode_mag(m, c) for c in range(1 << m)]
        assert sum(1 for v in vals if 2.0 ** (i - 1) <= v < 2.0 ** i) == (1 << k)
    assert orc.decode_mag(m, (1 << m) - 1) == 2.0 ** (m - 1)


@pytest.mark.parametrize("m", ALL_M)
def test_decoder_fields_reproduce_the_value(m):
    for c in range(1 << (m - 1), 1 << m):       # start bit 1
        e, man = orc.decode_fields(m, c)
        assert (man >> (m - 1)) == 1            # hidden one sits in the MSB
        assert Fraction(orc.decode_mag(m, c)) == Fraction(man, 1 << (m - 1)) * Fraction(2) ** e


@pytest.mark.parametrize("bits", range(2, 9))
def test_signed_format_is_sign_plus_magnitude(bits):
    m = bits - 1
    tab = orc.decode_table(bits, True)
    assert tab.shape == (1 << bits,)
    for c in range(1 << m):
        assert tab[c] == orc.decode_mag(m, c)
        assert tab[(1 << m) | c] == -orc.decode_mag(m, c) or c == 0
    assert tab[1 << m] == 0.0 and not np.signbit(tab[1 << m])
    # exactly one redundant pattern: 2^bits - 1 distinct values
    assert len(set(tab.tolist())) == (1 << bits) - 1
    # sign-magnitude order is strictly monotone
    order = [(1 << m) | c for c in range((1 << m) - 1, 0, -1)] + list(range(1 << m))
    vals = [tab[c] for c in order]
    assert all(b > a for a, b in zip(vals, vals[1:]))


@pytest.mark.parametrize("bits", range(2, 9))
def test_unsigned_table_matches_magnitude(bits):
    tab = orc.decode_table(bits, False)
    assert [orc.decode_mag(bits, c) for c in range(1 << bits)] == tab.tolist()


def test_container_fit_table():
    # (m, max integer image, max significant bits) from enumerating the format
    want = {1: (1, 1), 2: (4, 1), 3: (16, 2), 4: (64, 3), 5: (256, 4),
            6: (1024, 5), 7: (4096, 6), 8: (16384, 7)}
    for m, (imax, sig) in want.items():
        ints = [int(Fraction(orc.decode_mag(m, c)) * 2 ** (m - 1)) for c in range(1 << m)]
        assert max(ints) == imax
        worst = 0
        for n in ints:
            if n:
                while n % 2 == 0:
                    n //= 2
                worst = max(worst, n.bit_length())
        assert worst == sig
