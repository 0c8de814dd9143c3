"""Pins for the oracle's RMSE metric (Eq. 2): numpy fp64 on separately quantized data, closed forms and invariants."""
import numpy as np
import pytest

from oracle import dybit_oracle as orc


@pytest.mark.parametrize("fmt", [(4, True), (4, False), (8, True), (2, True), (6, False)])
def test_rmse_against_numpy(fmt):
    rng = np.random.default_rng(fmt[0])
    x = rng.normal(0.3, 1.7, 5001).astype(np.float32)
    if not fmt[1]:
        x = np.abs(x)
    sp = orc.absmax_scale(x, *fmt)
    xhat = orc.dequantize(orc.quantize(x, fmt[0], fmt[1], sp[1]), fmt[0], fmt[1], sp[0]).astype(np.float64)
    x64 = x.astype(np.float64)
    sigma = np.std(x64)                                  # population standard deviation
    want = np.sqrt(np.mean(((x64 - xhat) / sigma) ** 2))
    got, got_sigma, got_mse = orc.rmse(x, fmt[0], fmt[1], sp)
    assert got == pytest.approx(want, rel=1e-12)
    assert got_sigma == pytest.approx(sigma, rel=1e-12)
    assert got_mse == pytest.approx(np.mean((x64 - xhat) ** 2), rel=1e-12)


def test_rmse_closed_forms():
    # representable values quantize without error
    tab = orc.decode_table(4, True).astype(np.float32)
    assert orc.rmse(tab, 4, True, (1.0, 1.0))[0] == 0.0
    # two points +-0.375 in unsigned-magnitude terms sit exactly half-way between 0.25 and 0.5 (signed 4-bit, m = 3):
    # every error is 0.125, sigma is 0.375 -> RMSE = 1/3
    x = np.array([0.375, -0.375] * 8, dtype=np.float32)
    r, sigma, mse = orc.rmse(x, 4, True, (1.0, 1.0))
    assert sigma == pytest.approx(0.375) and mse == pytest.approx(0.125 ** 2) and r == pytest.approx(1.0 / 3.0)
    # degenerate tensors
    assert orc.rmse(np.zeros(0, np.float32), 4, True, (1.0, 1.0))[0] == 0.0
    assert orc.rmse(np.full(7, 0.3, np.float32), 4, True, (1.0, 1.0))[0] == 0.0      # sigma == 0


def test_rmse_is_invariant_under_power_of_two_rescaling_and_falls_with_bits():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 1, 4000).astype(np.float32)
    sp = orc.absmax_scale(x, 4, True)
    sp8 = orc.absmax_scale(x * 8, 4, True)
    assert orc.rmse(x, 4, True, sp)[0] == pytest.approx(orc.rmse(x * 8, 4, True, sp8)[0], rel=1e-12)
    errs = [orc.rmse(x, b, True, orc.absmax_scale(x, b, True))[0] for b in (2, 3, 4, 5, 6, 7, 8)]
    assert all(b < a for a, b in zip(errs, errs[1:]))
