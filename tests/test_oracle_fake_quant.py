"""Pins for the oracle's fake-quantization pair (QAT forward, clipped straight-through backward)."""
import numpy as np
import pytest

from oracle import dybit_oracle as orc


def _table1_unsigned4():
    vals = []
    for line in open(__file__.rsplit("/", 1)[0] + "/golden/table1_unsigned4.txt"):
        line = line.split("#")[0].strip()
        if line:
            vals.append(float(line.split()[-1]))
    return np.array(vals, dtype=np.float32)


def test_forward_fixes_the_values_the_paper_tabulates():
    # every value of the printed 4-bit unsigned table is its own image, at scale 1 and at a power-of-two scale
    tab = _table1_unsigned4()
    assert np.array_equal(orc.fake_quant(tab, 4, False, (1.0, 1.0)), tab)
    assert np.array_equal(orc.fake_quant(tab * 0.25, 4, False, (0.25, 4.0)), tab * 0.25)


def test_forward_hand_worked_example_signed_4bit():
    # signed 4-bit, m = 3: magnitudes 0, .25, .5, .75, 1, 1.5, 2, 4 (Eq. 1).  Nearest value; ties to the even code.
    x = np.array([0.1, 0.13, -0.3, 0.62, -0.9, 1.2, 1.76, -2.9, 3.1, 100.0, -7.0, 0.0], dtype=np.float32)
    want = np.array([0.0, 0.25, -0.25, 0.5, -1.0, 1.0, 2.0, -2.0, 4.0, 4.0, -4.0, 0.0], dtype=np.float32)
    assert np.array_equal(orc.fake_quant(x, 4, True, (1.0, 1.0)), want)
    # same numbers under scale 0.5: inputs and outputs halve
    assert np.array_equal(orc.fake_quant(x * 0.5, 4, True, (0.5, 2.0)), want * 0.5)


@pytest.mark.parametrize("fmt", [(2, True), (3, False), (4, True), (5, False), (8, True), (8, False)])
def test_forward_is_idempotent_nearest_and_inside_the_table(fmt):
    rng = np.random.default_rng(fmt[0])
    x = rng.laplace(0.0, 1.0, 4000).astype(np.float32)
    sp = orc.absmax_scale(x, *fmt)
    y = orc.fake_quant(x, fmt[0], fmt[1], sp)
    assert np.array_equal(orc.fake_quant(y, fmt[0], fmt[1], sp), y)
    grid = (np.float32(sp[0]) * orc.decode_table(*fmt).astype(np.float32)).astype(np.float64)
    assert np.isin(y.astype(np.float64), grid).all()
    # no grid point is closer to x than the image (brute force over the whole table, fp64; t = x * inv is
    # rounded to fp32 before the comparison, hence the small slack)
    d_img = np.abs(x.astype(np.float64) - y)
    d_best = np.abs(x.astype(np.float64)[:, None] - grid[None, :]).min(axis=1)
    assert (d_img <= d_best + 1e-6 * np.abs(x) + 1e-30).all()


def test_backward_hand_worked_masks():
    g = np.arange(1, 9, dtype=np.float32)
    x = np.array([-5.0, -4.0, -0.1, 0.0, 0.3, 4.0, 4.0000005, np.nan], dtype=np.float32)
    # signed 4-bit at scale 1 covers [-4, 4], ends included
    assert orc.fake_quant_backward(x, g, 4, True, (1.0, 1.0)).tolist() == [0, 2, 3, 4, 5, 6, 0, 0]
    # unsigned 4-bit at scale 0.5 covers [0, 4] (largest value 8 * 0.5)
    assert orc.fake_quant_backward(x, g, 4, False, (0.5, 2.0)).tolist() == [0, 0, 0, 4, 5, 6, 0, 0]
    # unsigned 2-bit at scale 1 covers [0, 2]
    assert orc.fake_quant_backward(x, g, 2, False, (1.0, 1.0)).tolist() == [0, 0, 0, 4, 5, 0, 0, 0]


@pytest.mark.parametrize("fmt", [(4, True), (3, False), (8, True)])
def test_backward_agrees_with_where_the_forward_is_flat(fmt):
    # outside the covered range the forward is constant (its finite difference is 0) and the gradient is cut;
    # with the max-abs scale nothing lies outside and the gradient passes untouched
    rng = np.random.default_rng(7)
    x = rng.normal(0.0, 1.0, 3000).astype(np.float32)
    if not fmt[1]:
        x = np.abs(x)
    g = rng.normal(0.0, 1.0, 3000).astype(np.float32)
    sp = orc.absmax_scale(x, *fmt)
    assert np.array_equal(orc.fake_quant_backward(x, g, fmt[0], fmt[1], sp), g)
    tight = (np.float32(sp[0]) * np.float32(0.25), np.float32(1.0) / (np.float32(sp[0]) * np.float32(0.25)))
    gx = orc.fake_quant_backward(x, g, fmt[0], fmt[1], tight)
    cut = gx == 0
    assert cut.any() and (~cut).any()
    eps = np.float32(1e-3)
    flat = orc.fake_quant(x + eps, fmt[0], fmt[1], tight) == orc.fake_quant(x - eps, fmt[0], fmt[1], tight)
    hi = float(tight[0]) * 2.0 ** (fmt[0] - (1 if fmt[1] else 0) - 1)
    far = np.abs(x) > hi * 1.01
    assert (cut[far]).all() and flat[far].all()
    assert np.array_equal(gx[~cut], g[~cut])
