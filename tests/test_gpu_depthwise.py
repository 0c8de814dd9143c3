"""GPU parity of the depth-wise convolution against the oracle.

Formats with at most 4 magnitude bits on both sides: bit-exact fp32.  Wider formats accumulate products beyond
2^24 in fp32: |err| <= 1e-5 * r*s * max|x| * max|w|.
"""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_dw(n, h, w, c, r, s, stride, pad, dil, fx, fw, seed=0):
    x = wl.half_normal((n, h, w, c), seed=seed) if not fx[1] else wl.normal((n, h, w, c), seed=seed)
    wt = wl.normal((c, r * s), seed=seed + 1, std=0.3)
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx)
    pw, sw = dy.dybit_quantize_pack_2d(wt.to(DEV), fw)
    spx = orc.absmax_scale(x.numpy(), fx[0], bool(fx[1]))
    spw = orc.absmax_scale(wt.numpy(), fw[0], bool(fw[1]))
    cx = orc.quantize(x.numpy(), fx[0], bool(fx[1]), spx[1])
    cw = orc.quantize(wt.numpy(), fw[0], bool(fw[1]), spw[1]).reshape(c, r, s)
    desc = dy.ConvDesc(n, h, w, c, c, r, s, stride, pad, dil)
    Y = dy.dybit_depthwise_conv2d(desc, px, fx, sx, pw, fw, sw)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    _, y_ref = orc.depthwise_conv2d(cx, fx, spx[0], cw, fw, spw[0], stride, pad, dil)
    got = Y.cpu().numpy()
    assert got.shape == y_ref.shape
    mx, mw = fx[0] - fx[1], fw[0] - fw[1]
    if mx <= 4 and mw <= 4:
        assert np.array_equal(got, y_ref)
    else:
        amax = float(spx[0]) * float(np.abs(orc.decode_table(fx[0], bool(fx[1]))).max())
        bmax = float(spw[0]) * float(np.abs(orc.decode_table(fw[0], bool(fw[1]))).max())
        tol = 1e-5 * r * s * amax * bmax
        assert np.abs(got.astype(np.float64) - y_ref.astype(np.float64)).max() <= tol


# MobileNetV2 depth-wise shapes at batch 2 (channels, input size, stride), 4-bit activations and weights
@pytest.mark.parametrize("c,hw,stride", [(32, 112, 1), (96, 112, 2), (144, 56, 1), (144, 56, 2), (192, 28, 1),
                                         (192, 28, 2), (384, 14, 1), (576, 14, 2), (960, 7, 1)])
def test_mobilenetv2_shapes_4bit(c, hw, stride):
    run_dw(2, hw, hw, c, 3, 3, stride, 1, 1, (4, 0), (4, 1), seed=c + stride)


@pytest.mark.parametrize("fx,fw", [((2, 0), (2, 1)), ((3, 0), (5, 1)), ((5, 1), (3, 1)), ((8, 0), (4, 1)), ((4, 1), (4, 1)),
                                   ((6, 0), (2, 1)), ((8, 0), (8, 1)), ((7, 1), (6, 1)), ((5, 0), (8, 1))])
def test_all_decode_paths_and_wide_formats(fx, fw):
    # 48 channels: word-aligned pixels for 2/4/8 bits, byte-wise extraction for the rest; ragged tiles
    run_dw(3, 13, 11, 48, 3, 3, 1, 1, 1, fx, fw, seed=fx[0] * 9 + fw[0])


@pytest.mark.parametrize("n,h,w,c,r,s,stride,pad,dil", [
    (1, 1, 1, 1, 1, 1, 1, 0, 1),          # a single code
    (2, 9, 9, 5, 3, 3, 1, 1, 1),          # 5 channels: pixels are not byte-aligned for 4-bit codes
    (1, 17, 15, 40, 5, 5, 1, 2, 1),       # 5x5 filter (generic loop), channels not a multiple of 32
    (2, 16, 16, 24, 3, 3, 1, 2, 2),       # dilation 2
    (1, 20, 18, 16, 3, 1, 3, 0, 1),       # stride 3, 3x1 filter, no padding
    (2, 8, 8, 72, 7, 7, 2, 3, 1),         # 7x7 stride 2
    (1, 5, 40, 64, 1, 3, 1, 1, 1),        # padding taller than the filter: all-padding rows
])
def test_edge_geometries(n, h, w, c, r, s, stride, pad, dil):
    run_dw(n, h, w, c, r, s, stride, pad, dil, (4, 0), (4, 1), seed=h * w + c)
    run_dw(n, h, w, c, r, s, stride, pad, dil, (3, 1), (4, 1), seed=h * w + c + 1)


def test_argument_errors():
    one = torch.tensor([1.0, 1.0], device=DEV)
    X = torch.zeros(64, dtype=torch.uint8, device=DEV)
    W = torch.zeros((8, 16), dtype=torch.uint8, device=DEV)
    with pytest.raises(Exception):                       # k != c
        dy.dybit_depthwise_conv2d(dy.ConvDesc(1, 4, 4, 8, 16, 3, 3, 1, 1, 1), X, (4, 0), one, W, (4, 1), one)
    with pytest.raises(Exception):                       # format
        dy.dybit_depthwise_conv2d(dy.ConvDesc(1, 4, 4, 8, 8, 3, 3, 1, 1, 1), X, (9, 0), one, W, (4, 1), one)
    with pytest.raises(Exception):                       # weight rows too short for 7x7 taps of 8-bit codes
        dy.dybit_depthwise_conv2d(dy.ConvDesc(1, 4, 4, 8, 8, 7, 7, 1, 3, 1), X, (4, 0), one, W, (8, 1), one)
