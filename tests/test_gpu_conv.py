"""GPU parity: dybit_conv2d (implicit GEMM) against the oracle's direct convolution."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_conv(layer, fx, fw, seed=0):
    """Quantize synthetic NHWC activations / KRSC weights on the GPU, convolve, compare with the oracle."""
    x = wl.half_normal((layer.n, layer.h, layer.w, layer.c), seed=seed)
    if fx[1]:
        x = x - 0.5
    w = wl.kaiming_normal(layer.k, layer.r, layer.s, layer.c, seed=seed + 1)
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(layer.k, -1).to(DEV), fw)
    spx = orc.absmax_scale(x.numpy(), fx[0], bool(fx[1]))
    spw = orc.absmax_scale(w.numpy(), fw[0], bool(fw[1]))
    cx = orc.quantize(x.numpy(), fx[0], bool(fx[1]), spx[1])
    cw = orc.quantize(w.numpy(), fw[0], bool(fw[1]), spw[1])
    assert np.array_equal(px.cpu().numpy(), orc.pack(cx, fx[0]))
    assert np.array_equal(pw.cpu().numpy(), orc.pack_rows(cw.reshape(layer.k, -1), fw[0]))
    desc = dy.ConvDesc(layer.n, layer.h, layer.w, layer.c, layer.k, layer.r, layer.s, layer.stride, layer.pad, 1)
    cont, _, _ = dy.dybit_choose_container(fx, fw)
    Y, Y_raw = dy.dybit_conv2d(desc, px, fx, sx, pw, fw, sw, want_raw=(cont == 0))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    S, Y_ref = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=layer.stride, pad=layer.pad)
    assert tuple(Y.shape) == Y_ref.shape
    if cont == 0:
        assert np.array_equal(Y_raw.cpu().numpy().astype(np.int64), S)
        assert np.array_equal(Y.cpu().numpy(), Y_ref)
    else:
        amax = float(spx[0]) * float(np.abs(orc.decode_table(fx[0], bool(fx[1]))).max())
        bmax = float(spw[0]) * float(np.abs(orc.decode_table(fw[0], bool(fw[1]))).max())
        tol = 1e-5 * layer.gemm_k * amax * bmax
        err = np.abs(Y.cpu().numpy().astype(np.float64) - Y_ref.astype(np.float64)).max()
        assert err <= tol, (err, tol)
    return cont


def _distinct_shapes(layers):
    seen, out = set(), []
    for L in layers:
        key = (L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad)
        if key not in seen:
            seen.add(key)
            out.append(L)
    return out


@pytest.mark.parametrize("layer", _distinct_shapes(wl.resnet18_layers(2)), ids=lambda L: L.name)
def test_resnet18_shapes_batch2_uniform_4bit(layer):
    # every distinct ResNet-18 layer shape, weights signed 4-bit, activations unsigned 4-bit
    assert run_conv(layer, (4, 0), (4, 1), seed=hash(layer.name) % 1000) == 0


@pytest.mark.parametrize("fx,fw", [((2, 0), (2, 1)), ((3, 0), (5, 1)), ((5, 0), (4, 1)), ((6, 0), (3, 1)),
                                   ((8, 0), (8, 1)), ((4, 1), (6, 1))])
def test_mixed_bitwidths_small_conv(fx, fw):
    L = wl.ConvLayer("t", 2, 14, 14, 64, 96, 3, 3, 1, 1)
    run_conv(L, fx, fw, seed=fx[0] * 10 + fw[0])


@pytest.mark.parametrize("shape", [
    wl.ConvLayer("stride2_3x3_ragged", 3, 15, 13, 32, 40, 3, 3, 2, 1),
    wl.ConvLayer("pointwise_stride2", 2, 9, 9, 48, 130, 1, 1, 2, 0),
    wl.ConvLayer("c3_7x7", 1, 32, 32, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c20_pad_channels", 2, 8, 8, 20, 24, 3, 3, 1, 1),
    wl.ConvLayer("fc_like", 5, 1, 1, 512, 1000, 1, 1, 1, 0),
    wl.ConvLayer("one_pixel", 1, 1, 1, 16, 1, 1, 1, 1, 0),
    wl.ConvLayer("gather_long_k_c48_7x7", 2, 12, 12, 48, 40, 7, 7, 1, 3),
    wl.ConvLayer("gather_long_k_c128_small_image", 1, 10, 10, 128, 64, 3, 3, 2, 1),
], ids=lambda L: L.name)
def test_edge_geometries(shape):
    assert run_conv(shape, (4, 0), (4, 1), seed=3) == 0


# Large enough activations that the TMA im2col path is taken (>= 128 KiB expanded), for both swizzle
# spans (64-byte pixels and multiples of 128 bytes), strides, dilation, ragged last tile.
@pytest.mark.parametrize("shape,fx,fw", [
    (wl.ConvLayer("c64_3x3_s1", 8, 28, 28, 64, 64, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c64_3x3_s2_ragged", 5, 29, 27, 64, 72, 3, 3, 2, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c64_1x1_s2", 6, 28, 28, 64, 128, 1, 1, 2, 0), (4, 0), (4, 1)),
    (wl.ConvLayer("c128_3x3_s1", 6, 20, 20, 128, 96, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c256_3x3_s2", 8, 14, 14, 256, 256, 3, 3, 2, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c512_3x3_s1", 8, 7, 7, 512, 512, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c256_1x1_s2", 8, 14, 14, 256, 512, 1, 1, 2, 0), (3, 0), (2, 1)),
    (wl.ConvLayer("c128_5x5_pad2", 4, 18, 18, 128, 40, 5, 5, 1, 2), (4, 1), (4, 1)),
    (wl.ConvLayer("c64_bf16", 6, 20, 20, 64, 96, 3, 3, 1, 1), (8, 0), (8, 1)),
    (wl.ConvLayer("c128_e4m3", 6, 20, 20, 128, 96, 3, 3, 2, 1), (5, 0), (4, 1)),
    (wl.ConvLayer("c32_bf16_64B_pixels", 8, 24, 24, 32, 48, 3, 3, 1, 1), (6, 0), (8, 1)),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_im2col_tma_path(shape, fx, fw):
    run_conv(shape, fx, fw, seed=11)


@pytest.mark.parametrize("shape", [
    wl.ConvLayer("pw_c64", 4, 28, 28, 64, 256, 1, 1, 1, 0),
    wl.ConvLayer("pw_c256_ragged", 3, 13, 11, 256, 100, 1, 1, 1, 0),
    wl.ConvLayer("pw_c48", 2, 9, 9, 48, 64, 1, 1, 1, 0),
], ids=lambda L: L.name)
def test_pointwise_conv_runs_as_plain_gemm(shape):
    run_conv(shape, (4, 0), (4, 1), seed=5)
    run_conv(shape, (8, 0), (6, 1), seed=6)


# at most four one-byte channels: pixels as 32-bit words gathered by the tensor-core kernel (no patch matrix);
# two-byte elements (6 or more magnitude bits) take the patch-matrix path instead
@pytest.mark.parametrize("shape", [
    wl.ConvLayer("c3_7x7_s2_ragged", 2, 37, 41, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c3_3x3", 3, 19, 23, 3, 40, 3, 3, 1, 1),
    wl.ConvLayer("c1_5x5_s2", 2, 30, 28, 1, 24, 5, 5, 2, 2),
    wl.ConvLayer("c2_8x8_nopad", 1, 26, 26, 2, 72, 8, 8, 1, 0),
    wl.ConvLayer("c4_9x3_s3", 2, 33, 21, 4, 130, 9, 3, 3, 1),
    wl.ConvLayer("c3_1x7", 2, 12, 40, 3, 16, 1, 7, 1, 3),
], ids=lambda L: L.name)
@pytest.mark.parametrize("fx,fw", [((4, 0), (4, 1)), ((3, 1), (2, 1)), ((5, 0), (4, 1)), ((8, 0), (4, 1))])
def test_few_channel_geometries(shape, fx, fw):
    run_conv(shape, fx, fw, seed=len(shape.name) + fx[0])


# Stride-1 convolutions with up to three filter rows and pixels of 64 / k*128 container bytes run on halo tiles
# (th x 8 output pixels of ni images): geometries that exercise clipped tile rows and columns, several images per
# tile with an odd batch, one to three filter rows, wide filters, zero and large padding, several channel blocks,
# several tile columns of output channels, and all three containers.
@pytest.mark.parametrize("shape,fx,fw", [
    (wl.ConvLayer("h56_c64_k64", 2, 56, 56, 64, 64, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("h7_two_images_per_tile_odd_batch", 5, 7, 7, 128, 72, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("h4_three_images_per_tile", 7, 4, 5, 64, 40, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("h30_w19_ragged", 3, 30, 19, 64, 200, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("h17_nopad", 2, 17, 21, 128, 96, 3, 3, 1, 0), (4, 0), (4, 1)),
    (wl.ConvLayer("r1_s3", 2, 12, 20, 64, 48, 1, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("r2_s2_pad1", 3, 9, 9, 128, 64, 2, 2, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("r3_s5_pad2", 2, 14, 14, 64, 300, 3, 5, 1, 2), (4, 0), (4, 1)),
    (wl.ConvLayer("c384_three_channel_blocks", 2, 14, 14, 384, 128, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("c512_k512_h7", 4, 7, 7, 512, 512, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("bf16_c64", 3, 14, 14, 64, 96, 3, 3, 1, 1), (8, 0), (8, 1)),
    (wl.ConvLayer("e4m3_c128", 3, 14, 14, 128, 96, 3, 3, 1, 1), (5, 0), (4, 1)),
    (wl.ConvLayer("k_not_multiple_of_4_falls_back", 2, 14, 14, 64, 70, 3, 3, 1, 1), (4, 0), (4, 1)),
    (wl.ConvLayer("pad3_larger_than_filter", 2, 10, 10, 64, 64, 3, 3, 1, 3), (4, 0), (4, 1)),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_halo_tile_path(shape, fx, fw):
    dy.dybit_set_conv_lowering(1)            # halo tiles wherever they apply, not only where they are the default
    try:
        run_conv(shape, fx, fw, seed=23)
    finally:
        dy.dybit_set_conv_lowering(0)


def test_conv_lowerings_agree_bit_for_bit():
    # the same convolution through the default choice, forced halo tiles and no halo tiles: identical outputs
    L = wl.ConvLayer("c64_k64", 4, 28, 28, 64, 64, 3, 3, 1, 1)
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=5)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=6)
    px, sx = dy.dybit_quantize_pack(x.to(DEV), (4, 0))
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), (4, 1))
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, 1, 1, 1)
    outs = []
    try:
        for mode in (0, 1, 2):
            dy.dybit_set_conv_lowering(mode)
            Y, Y_raw = dy.dybit_conv2d(desc, px, (4, 0), sx, pw, (4, 1), sw, want_raw=True)
            outs.append((Y.clone(), Y_raw.clone()))
    finally:
        dy.dybit_set_conv_lowering(0)
    with pytest.raises(dy.DybitError):
        dy.dybit_set_conv_lowering(3)
    for Y, Y_raw in outs[1:]:
        assert torch.equal(Y, outs[0][0]) and torch.equal(Y_raw, outs[0][1])


# Stride-2 convolutions on at most four one-byte channels with even image sides (the 7 x 7 stem) run on a 2 x 2
# space-to-depth image with halo tiles: every filter size / padding that fits four rearranged taps, 1-4 channels,
# output channel counts the TMA store cannot take (direct stores), several tile rows and columns, odd batch.
@pytest.mark.parametrize("shape", [
    wl.ConvLayer("stem_7x7_p3", 3, 64, 48, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("stem_7x7_p3_c4", 2, 32, 32, 4, 64, 7, 7, 2, 3),
    wl.ConvLayer("c1_5x5_p2", 2, 30, 28, 1, 24, 5, 5, 2, 2),
    wl.ConvLayer("c2_3x3_p1", 5, 20, 36, 2, 40, 3, 3, 2, 1),
    wl.ConvLayer("c3_4x4_p0", 2, 18, 22, 3, 128, 4, 4, 2, 0),
    wl.ConvLayer("c3_2x2_p0", 2, 16, 16, 3, 16, 2, 2, 2, 0),
    wl.ConvLayer("c3_6x6_p2_k70_direct_stores", 2, 24, 24, 3, 70, 6, 6, 2, 2),
    wl.ConvLayer("c3_7x7_p3_k200_two_tile_columns", 1, 40, 40, 3, 200, 7, 7, 2, 3),
], ids=lambda L: L.name)
@pytest.mark.parametrize("fx,fw", [((4, 0), (4, 1)), ((5, 0), (4, 1)), ((2, 1), (3, 1))])
def test_space_to_depth_stem_path(shape, fx, fw):
    run_conv(shape, fx, fw, seed=len(shape.name) + fw[0])
