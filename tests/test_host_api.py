"""CPU-only checks of the C-ABI library: it loads, exports every declared
symbol, and its host-side logic (Eq. 1 enumeration, container choice, size
helpers, argument validation) agrees with the oracle and with the format's
definition.  No kernel is launched here."""
import ctypes
import os
import re
from fractions import Fraction

import numpy as np
import pytest

import paper_2302_12510_b200 as dy
from oracle import dybit_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FORMATS = [(b, s) for b in range(2, 9) for s in (0, 1)]


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dybit.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(dybit_[a-z0-9_]+)\s*\(", header))
    assert {"dybit_quantize_pack", "dybit_decode", "dybit_gemm", "dybit_conv2d"} <= names
    raw = ctypes.CDLL(os.path.join(ROOT, "paper_2302_12510_b200", "libdybit.so"))
    for n in sorted(names):
        assert hasattr(raw, n), n
        assert hasattr(dy, n), f"python binding lacks {n}"


@pytest.mark.parametrize("fmt", FORMATS)
def test_decode_table_matches_oracle(fmt):
    got = np.array(dy.dybit_decode_table(fmt))
    want = orc.decode_table(fmt[0], bool(fmt[1]))
    assert np.array_equal(got[: 1 << fmt[0]], want)
    assert not got[1 << fmt[0]:].any()


def _narrowest(fmt):
    """Container class of one format from the oracle's table: 0 int8, 1 e4m3, 2 bf16."""
    vals = [Fraction(v) for v in orc.decode_table(fmt[0], bool(fmt[1]))]
    e = 0
    while any((v * 2 ** e).denominator != 1 for v in vals):
        e += 1
    if max(abs(v * 2 ** e) for v in vals) <= 127:
        return 0, e
    def sig(v):
        n = abs(v.numerator)
        while n and n % 2 == 0:
            n //= 2
        return n.bit_length()
    if all(sig(v) <= 4 and (v == 0 or Fraction(1, 512) <= abs(v) <= 448) for v in vals):
        return 1, 0
    assert all(sig(v) <= 8 for v in vals)
    return 2, 0


@pytest.mark.parametrize("fa", FORMATS)
@pytest.mark.parametrize("fb", [(4, 1), (4, 0), (6, 0), (8, 1), (2, 1)])
def test_container_choice_by_enumeration(fa, fb):
    ca, ea = _narrowest(fa)
    cb, eb = _narrowest(fb)
    cont, xa, xb = dy.dybit_choose_container(fa, fb)
    assert cont == max(ca, cb)
    if cont == 0:
        assert (xa, xb) == (ea, eb)
    else:
        assert (xa, xb) == (0, 0)


def test_size_helpers():
    for bits in range(2, 9):
        for n in (0, 1, 127, 128, 129, 1000, 2 ** 30):
            assert dy.dybit_packed_bytes(n, bits) == orc.packed_bytes(n, bits)
        for k in (1, 128, 129, 147, 4608):
            assert dy.dybit_row_stride_bytes(k, bits) == orc.row_stride_bytes(k, bits)
            assert dy.dybit_row_stride_bytes(k, bits) % 16 == 0
    assert dy.dybit_packed_bytes(10, 9) == 0 and dy.dybit_packed_bytes(-1, 4) == 0
    assert dy.dybit_row_stride_bytes(0, 4) == 0


def test_conv_output_size():
    assert dy.dybit_conv2d_out_hw(dy.ConvDesc(1, 224, 224, 3, 64, 7, 7, 2, 3, 1)) == (112, 112)
    assert dy.dybit_conv2d_out_hw(dy.ConvDesc(1, 56, 56, 64, 128, 3, 3, 2, 1, 1)) == (28, 28)
    assert dy.dybit_conv2d_out_hw(dy.ConvDesc(1, 56, 56, 64, 128, 1, 1, 2, 0, 1)) == (28, 28)
    with pytest.raises(dy.DybitError):
        dy.dybit_conv2d_out_hw(dy.ConvDesc(1, 2, 2, 3, 4, 5, 5, 1, 0, 1))


def test_status_strings_and_argument_errors():
    assert dy.dybit_status_string(0) == "ok"
    assert "workspace" in dy.dybit_status_string(4)
    L = dy.lib
    f4 = dy.binding._CFmt(4, 1)
    bad = dy.binding._CFmt(9, 0)
    # argument checks run before anything touches the device
    assert L.dybit_quantize_pack(None, 16, f4, None, None, None, None) == 1
    assert L.dybit_quantize_pack(ctypes.c_void_p(16), 16, bad, ctypes.c_void_p(16), ctypes.c_void_p(16), None, None) == 1
    assert L.dybit_quantize_pack(ctypes.c_void_p(16), 16, f4, ctypes.c_void_p(16), ctypes.c_void_p(24), None, None) == 3
    assert L.dybit_quantize_pack_2d(ctypes.c_void_p(16), 4, 300, 200, f4, ctypes.c_void_p(16), ctypes.c_void_p(16),
                                    192, None, None) == 1            # ld < cols
    assert L.dybit_quantize_pack_2d(ctypes.c_void_p(16), 4, 300, 300, f4, ctypes.c_void_p(16), ctypes.c_void_p(16),
                                    128, None, None) == 1            # stride too small
    assert L.dybit_decode(None, 5, f4, None, None, None) == 1
    assert L.dybit_absmax_scale(ctypes.c_void_p(16), -1, f4, ctypes.c_void_p(16), None) == 1
    with pytest.raises(dy.DybitError):
        dy.dybit_decode_table((1, 0))
    with pytest.raises(dy.DybitError):
        dy.dybit_choose_container((4, 1), (12, 0))
