"""GPU parity of dybit_quantize_conv2d (fp32 activation in, codes + layer output out) against the oracle: the codes
and the scale must be those of the oracle's quantizer, the output that of the oracle's convolution on those codes."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run(layer, fx, fw, seed=0, given_scale=False):
    x = wl.half_normal((layer.n, layer.h, layer.w, layer.c), seed=seed)
    if fx[1]:
        x = x - 0.5
    w = wl.kaiming_normal(layer.k, layer.r, layer.s, layer.c, seed=seed + 1)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(layer.k, -1).to(DEV), fw)
    spw = orc.absmax_scale(w.numpy(), fw[0], bool(fw[1]))
    cw = orc.quantize(w.numpy(), fw[0], bool(fw[1]), spw[1])
    if given_scale:
        # a calibrated scale below the maximum: the largest activations saturate
        full = orc.absmax_scale(x.numpy(), fx[0], bool(fx[1]))
        s0 = np.float32(full[0]) * np.float32(0.6)
        spx = (float(s0), float(np.float32(1.0) / s0))
        scale_x = torch.tensor(spx, dtype=torch.float32, device=DEV)
    else:
        spx = orc.absmax_scale(x.numpy(), fx[0], bool(fx[1]))
        scale_x = None
    cx = orc.quantize(x.numpy(), fx[0], bool(fx[1]), spx[1])
    desc = dy.ConvDesc(layer.n, layer.h, layer.w, layer.c, layer.k, layer.r, layer.s, layer.stride, layer.pad, 1)
    cont, _, _ = dy.dybit_choose_container(fx, fw)
    Y, Y_raw, packed, scale = dy.dybit_quantize_conv2d(desc, x.to(DEV), fx, pw, fw, sw, scale_x=scale_x,
                                                       want_raw=(cont == 0))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    assert scale.cpu().numpy().tolist() == [float(np.float32(spx[0])), float(np.float32(spx[1]))]
    assert np.array_equal(packed.cpu().numpy(), orc.pack(cx, fx[0]))
    S, Y_ref = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=layer.stride, pad=layer.pad)
    if cont == 0:
        assert np.array_equal(Y_raw.cpu().numpy().astype(np.int64), S)
        assert np.array_equal(Y.cpu().numpy(), Y_ref)
    else:
        amax = float(spx[0]) * float(np.abs(orc.decode_table(fx[0], bool(fx[1]))).max())
        bmax = float(spw[0]) * float(np.abs(orc.decode_table(fw[0], bool(fw[1]))).max())
        err = np.abs(Y.cpu().numpy().astype(np.float64) - Y_ref.astype(np.float64)).max()
        assert err <= 1e-5 * layer.gemm_k * amax * bmax
    # and the two-call path gives the same bits
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx, scale=scale_x)
    Y2, _ = dy.dybit_conv2d(desc, px, fx, sx, pw, fw, sw)
    assert np.array_equal(Y.cpu().numpy().view(np.uint32), Y2.cpu().numpy().view(np.uint32))
    return cont


# one launch for codes + elements + weights: im2col (64-byte and 128-byte pixels), pointwise, cp.async gather
@pytest.mark.parametrize("layer", [
    wl.ConvLayer("c64_3x3_im2col", 8, 28, 28, 64, 64, 3, 3, 1, 1),
    wl.ConvLayer("c128_3x3_s2_im2col", 6, 20, 20, 128, 96, 3, 3, 2, 1),
    wl.ConvLayer("c256_pointwise_ragged", 3, 13, 11, 256, 100, 1, 1, 1, 0),
    wl.ConvLayer("c64_1x1_s2", 6, 28, 28, 64, 128, 1, 1, 2, 0),
    wl.ConvLayer("c48_gather", 2, 9, 9, 48, 64, 3, 3, 1, 1),
    wl.ConvLayer("c16_tiny", 1, 3, 5, 16, 8, 3, 3, 1, 1),
    wl.ConvLayer("fc_like", 5, 1, 1, 512, 1000, 1, 1, 1, 0),
], ids=lambda L: L.name)
def test_fused_layouts_4bit(layer):
    assert run(layer, (4, 0), (4, 1), seed=len(layer.name)) == 0
    assert run(layer, (4, 0), (4, 1), seed=len(layer.name) + 1, given_scale=True) == 0


# separate quantize + patch / padded expand: few channels, channels not a multiple of 16
@pytest.mark.parametrize("layer", [
    wl.ConvLayer("c3_7x7_patch", 2, 32, 32, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c20_pad_channels", 2, 8, 8, 20, 24, 3, 3, 1, 1),
], ids=lambda L: L.name)
def test_unfused_layouts(layer):
    assert run(layer, (4, 0), (4, 1), seed=3) == 0


@pytest.mark.parametrize("fx,fw,cont", [((2, 0), (2, 1), 0), ((3, 0), (5, 1), 0), ((5, 0), (4, 1), 1), ((6, 0), (3, 1), 2),
                                        ((8, 0), (8, 1), 2), ((4, 1), (6, 1), 1), ((7, 1), (2, 1), 2)])
def test_every_container_and_odd_widths(fx, fw, cont):
    L = wl.ConvLayer("t", 2, 14, 14, 64, 96, 3, 3, 1, 1)
    assert run(L, fx, fw, seed=fx[0] * 10 + fw[0]) == cont
    L = wl.ConvLayer("t_big", 6, 20, 20, 64, 96, 3, 3, 1, 1)       # large enough for the TMA im2col path
    assert run(L, fx, fw, seed=fx[0] * 10 + fw[0] + 1, given_scale=True) == cont


def test_resnet18_layer_at_bench_batch_sampled():
    L = [l for l in wl.resnet18_layers(32) if l.name == "layer2.0.conv2"][0]
    fx, fw = (4, 0), (4, 1)
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1, device=DEV)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    spw = orc.absmax_scale(w.numpy(), 4, True)
    cw = orc.quantize(w.numpy(), 4, True, spw[1])
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Y, _, packed, scale = dy.dybit_quantize_conv2d(desc, x, fx, pw, fw, sw)
    xh = x.cpu().numpy()
    spx = orc.absmax_scale(xh, 4, False)
    assert scale.cpu().numpy().tolist() == [float(np.float32(spx[0])), float(np.float32(spx[1]))]
    rng = np.random.default_rng(0)
    idx = np.concatenate([rng.integers(0, Y.numel(), 1500), [Y.numel() - 1]]).astype(np.int64)
    _, y_ref = orc.conv2d_sampled(xh, fx, spx, cw, fw, spw[0], idx, stride=L.stride, pad=L.pad)
    assert np.array_equal(Y.cpu().numpy().reshape(-1)[idx], y_ref)
    first = orc.pack(orc.quantize(xh.reshape(-1)[: 1 << 16], 4, False, spx[1]), 4)
    assert np.array_equal(packed.cpu().numpy()[: first.size], first)


def test_argument_errors():
    one = torch.tensor([1.0, 1.0], device=DEV)
    d = dy.ConvDesc(1, 4, 4, 16, 8, 3, 3, 1, 1, 1)
    W = torch.zeros((8, 80), dtype=torch.uint8, device=DEV)
    with pytest.raises(Exception):                       # wrong element count
        dy.dybit_quantize_conv2d(d, torch.zeros(100, device=DEV), (4, 0), W, (4, 1), one)
    with pytest.raises(Exception):                       # not fp32
        dy.dybit_quantize_conv2d(d, torch.zeros(256, device=DEV, dtype=torch.float16), (4, 0), W, (4, 1), one)


# few channels: the quantize launch writes one 32-bit word per pixel; element counts that are not multiples of
# the 1024-element chunk make pixels straddle chunk boundaries
@pytest.mark.parametrize("layer", [
    wl.ConvLayer("c3_7x7_s2_ragged", 2, 37, 41, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c3_stem_small", 2, 64, 64, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c1_5x5", 3, 30, 31, 1, 24, 5, 5, 1, 2),
    wl.ConvLayer("c2_3x3_s2", 5, 17, 29, 2, 48, 3, 3, 2, 1),
    wl.ConvLayer("c4_3x3", 2, 21, 21, 4, 32, 3, 3, 1, 1),
    wl.ConvLayer("c3_tiny", 1, 3, 5, 3, 8, 3, 3, 1, 1),
], ids=lambda L: L.name)
@pytest.mark.parametrize("fx,fw,given", [((4, 0), (4, 1), False), ((4, 1), (3, 1), True), ((5, 0), (5, 1), False),
                                         ((7, 0), (4, 1), False)])
def test_few_channels_pixel_words(layer, fx, fw, given):
    run(layer, fx, fw, seed=len(layer.name) * 3 + fx[0], given_scale=given)


def oracle_layer(layer, fx, fw, seed, given_scale):
    """Inputs of one layer and what the oracle makes of them."""
    x = wl.half_normal((layer.n, layer.h, layer.w, layer.c), seed=seed)
    if fx[1]:
        x = x - 0.5
    w = wl.kaiming_normal(layer.k, layer.r, layer.s, layer.c, seed=seed + 1)
    spw = orc.absmax_scale(w.numpy(), fw[0], bool(fw[1]))
    cw = orc.quantize(w.numpy(), fw[0], bool(fw[1]), spw[1])
    spx = orc.absmax_scale(x.numpy(), fx[0], bool(fx[1]))
    if given_scale:
        s0 = np.float32(spx[0]) * np.float32(0.7)
        spx = (float(s0), float(np.float32(1.0) / s0))
    cx = orc.quantize(x.numpy(), fx[0], bool(fx[1]), spx[1])
    S, Y_ref = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=layer.stride, pad=layer.pad)
    return x, w, spx, orc.pack(cx, fx[0]), S, Y_ref


# several independent layers through dybit_quantize_expand_layers + dybit_conv2d_prepared: one max-abs launch, one
# quantize + expand launch per pair of formats, then one tensor-core launch per layer (the few-channel patch lowering
# of the bf16 stem has a gather launch as well); results as the oracle's, layer by layer
def test_layers_in_few_launches():
    cases = [
        (wl.ConvLayer("stem_s2d", 2, 64, 64, 3, 64, 7, 7, 2, 3), (4, 0), (4, 1), False),
        (wl.ConvLayer("c64_3x3", 8, 28, 28, 64, 64, 3, 3, 1, 1), (4, 0), (4, 1), False),
        (wl.ConvLayer("c128_3x3_s2", 6, 20, 20, 128, 96, 3, 3, 2, 1), (4, 0), (4, 1), True),
        (wl.ConvLayer("c256_pointwise", 3, 13, 11, 256, 100, 1, 1, 1, 0), (4, 0), (4, 1), False),
        (wl.ConvLayer("c48_gather", 2, 9, 9, 48, 64, 3, 3, 1, 1), (4, 0), (4, 1), False),
        (wl.ConvLayer("fc_like", 5, 1, 1, 512, 1000, 1, 1, 1, 0), (4, 0), (4, 1), False),
        (wl.ConvLayer("c64_e4m3", 2, 14, 14, 64, 96, 3, 3, 1, 1), (5, 0), (4, 1), False),
        (wl.ConvLayer("c64_bf16", 6, 20, 20, 64, 96, 3, 3, 1, 1), (8, 0), (8, 1), True),
        (wl.ConvLayer("c1_5x5_signed", 3, 30, 31, 1, 24, 5, 5, 1, 2), (4, 1), (3, 1), False),
        (wl.ConvLayer("c64_3x3_again", 8, 28, 28, 64, 64, 3, 3, 1, 1), (4, 0), (4, 1), False),     # shares a launch with c64_3x3
    ]
    args, refs = [], []
    for i, (L, fx, fw, given) in enumerate(cases):
        x, w, spx, packed_ref, S, Y_ref = oracle_layer(L, fx, fw, 100 + 7 * i, given)
        pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
        cont, _, _ = dy.dybit_choose_container(fx, fw)
        a = dict(desc=dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1), X=x.to(DEV), fx=fx, W=pw, fw=fw,
                 scale_w=sw, want_raw=(cont == 0))
        if given:
            a["scale_x"] = torch.tensor(spx, dtype=torch.float32, device=DEV)
        args.append(a)
        refs.append((L, fx, fw, cont, spx, packed_ref, S, Y_ref, orc.absmax_scale(w.numpy(), fw[0], bool(fw[1]))))
    layers = dy.ConvLayers(args)
    torch.cuda.synchronize()
    n0 = dy.dybit_launch_count()
    dy.dybit_quantize_expand_layers(layers)
    n1 = dy.dybit_launch_count()
    assert n1 - n0 == 1 + 4                     # max-abs for all; (4,0)x(4,1), (5,0)x(4,1), (8,0)x(8,1), (4,1)x(3,1)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    for i in range(len(cases)):
        dy.dybit_conv2d_prepared(layers, i, stream=side if i % 2 else None)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert dy.dybit_launch_count() - n1 <= len(cases) + 2
    assert dy.dybit_last_device_status() == (0, 0)
    # the same tensor-core work through dybit_conv2d_prepared_layers (problems of one kernel configuration share a
    # launch): fewer launches, the same bits
    one_by_one = [(y.clone(), None if r is None else r.clone()) for y, r in zip(layers.Y, layers.raw)]
    for y in layers.Y:
        y.zero_()
    n2 = dy.dybit_launch_count()
    dy.dybit_conv2d_prepared_layers(layers)
    torch.cuda.synchronize()
    assert dy.dybit_launch_count() - n2 <= len(cases)      # one by one: a launch per layer + the patch gather of c48_gather
    assert dy.dybit_last_device_status() == (0, 0)
    for i, (y, r) in enumerate(one_by_one):
        assert torch.equal(y, layers.Y[i]), cases[i][0].name
        assert r is None or torch.equal(r, layers.raw[i]), cases[i][0].name
    for i, (L, fx, fw, cont, spx, packed_ref, S, Y_ref, spw) in enumerate(refs):
        assert layers.scale[i].cpu().numpy().tolist() == [float(np.float32(spx[0])), float(np.float32(spx[1]))], L.name
        assert np.array_equal(layers.packed[i].cpu().numpy(), packed_ref), L.name
        Y = layers.Y[i].cpu().numpy()
        if cont == 0:
            assert np.array_equal(layers.raw[i].cpu().numpy().astype(np.int64), S), L.name
            assert np.array_equal(Y, Y_ref), L.name
        else:
            amax = float(spx[0]) * float(np.abs(orc.decode_table(fx[0], bool(fx[1]))).max())
            bmax = float(spw[0]) * float(np.abs(orc.decode_table(fw[0], bool(fw[1]))).max())
            assert np.abs(Y.astype(np.float64) - Y_ref.astype(np.float64)).max() <= 1e-5 * L.gemm_k * amax * bmax, L.name
        # and bit for bit what the one-layer call gives
        a = args[i]
        Y1, _, p1, s1 = dy.dybit_quantize_conv2d(a["desc"], a["X"], fx, a["W"], fw, a["scale_w"], scale_x=a.get("scale_x"))
        assert np.array_equal(Y1.cpu().numpy().view(np.uint32), Y.view(np.uint32)), L.name
        assert torch.equal(p1, layers.packed[i]) and torch.equal(s1, layers.scale[i]), L.name


def test_layers_reject_a_lowering_without_fused_expand():
    # 120 channels: padded to 128 per tap and too long a row for the patch matrix, so quantize and expand stay apart
    L = wl.ConvLayer("c120_pad_channels", 2, 8, 8, 120, 24, 3, 3, 1, 1)
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1, device=DEV)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), (4, 1))
    layers = dy.ConvLayers([dict(desc=dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1), X=x, fx=(4, 0), W=pw,
                                 fw=(4, 1), scale_w=sw)])
    n0 = dy.dybit_launch_count()
    with pytest.raises(dy.DybitError):
        dy.dybit_quantize_expand_layers(layers)
    assert dy.dybit_launch_count() == n0
