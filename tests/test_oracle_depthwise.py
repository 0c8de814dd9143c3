"""Pins for the oracle's depth-wise convolution: the dense convolution with a block-diagonal filter bank, a
library correlation on the dequantized tensors, and a hand-worked case."""
import numpy as np
import pytest
from scipy.signal import correlate2d

from oracle import dybit_oracle as orc


def _codes(rng, shape, bits):
    return rng.integers(0, 1 << bits, size=shape, dtype=np.uint8)


@pytest.mark.parametrize("fx,fw,stride,pad,dil,r,s", [
    ((4, False), (4, True), 1, 1, 1, 3, 3),
    ((4, False), (4, True), 2, 1, 1, 3, 3),
    ((2, True), (3, True), 1, 2, 2, 3, 3),
    ((8, False), (8, True), 2, 0, 1, 5, 3),
    ((5, True), (2, True), 1, 0, 1, 1, 1),
])
def test_equals_dense_convolution_with_block_diagonal_filters(fx, fw, stride, pad, dil, r, s):
    rng = np.random.default_rng(r * 10 + s + stride)
    n, h, w, c = 2, 9, 8, 5
    cx = _codes(rng, (n, h, w, c), fx[0])
    cw = _codes(rng, (c, r, s), fw[0])
    # dense filter bank [k][r][s][c] that is zero (code 0) off the diagonal k == c
    dense = np.zeros((c, r, s, c), dtype=np.uint8)
    for ch in range(c):
        dense[ch, :, :, ch] = cw[ch]
    S_dw, y_dw = orc.depthwise_conv2d(cx, fx, 0.37, cw, fw, 0.011, stride, pad, dil)
    S_dn, y_dn = orc.conv2d(cx, fx, 0.37, dense, fw, 0.011, stride, pad, dil)
    assert np.array_equal(S_dw, S_dn)
    assert np.array_equal(y_dw, y_dn)


@pytest.mark.parametrize("fx,fw", [((4, False), (4, True)), ((3, True), (6, True)), ((8, True), (2, True))])
def test_against_scipy_correlation_of_the_dequantized_tensors(fx, fw):
    rng = np.random.default_rng(fx[0] + fw[0])
    n, h, w, c, r, s, pad = 2, 11, 7, 4, 3, 3, 1
    cx = _codes(rng, (n, h, w, c), fx[0])
    cw = _codes(rng, (c, r, s), fw[0])
    sx, sw = 0.5, 0.25                                    # powers of two: every product and sum below is exact
    xv = orc.dequantize(cx, fx[0], fx[1], sx).astype(np.float64)
    wv = orc.dequantize(cw, fw[0], fw[1], sw).astype(np.float64)
    _, y = orc.depthwise_conv2d(cx, fx, sx, cw, fw, sw, 1, pad, 1)
    for b in range(n):
        for ch in range(c):
            want = correlate2d(np.pad(xv[b, :, :, ch], pad), wv[ch], mode="valid")
            assert np.array_equal(y[b, :, :, ch].astype(np.float64), want)


def test_hand_worked_single_channel():
    # unsigned 4-bit input codes 8, 10, 12 decode to 1, 1.5, 2 (Table I); signed 4-bit weights 4, 12 are +1, -1
    tab = orc.decode_table(4, False)
    assert [tab[8], tab[10], tab[12]] == [1.0, 1.5, 2.0]
    wt = orc.decode_table(4, True)
    assert [wt[4], wt[12]] == [1.0, -1.0]
    x = np.array([8, 10, 12, 10], dtype=np.uint8).reshape(1, 1, 4, 1)           # 1 x 4 image: 1, 1.5, 2, 1.5
    k = np.array([12, 4], dtype=np.uint8).reshape(1, 1, 2)                    # kernel [-1, +1]: forward difference
    _, y = orc.depthwise_conv2d(x, (4, False), 1.0, k, (4, True), 1.0)
    assert y.reshape(-1).tolist() == [0.5, 0.5, -0.5]
    _, y = orc.depthwise_conv2d(x, (4, False), 2.0, k, (4, True), 0.5, stride=2)
    assert y.reshape(-1).tolist() == [0.5, -0.5]
    _, y = orc.depthwise_conv2d(x, (4, False), 1.0, k, (4, True), 1.0, pad=1)   # zero padding on both sides
    # the padding also adds a row above and below the 1 x 4 image: those output rows see zeros only
    assert y.shape == (1, 3, 5, 1)
    assert y[0, 1, :, 0].tolist() == [1.0, 0.5, 0.5, -0.5, -1.5]
    assert not y[0, 0].any() and not y[0, 2].any()
