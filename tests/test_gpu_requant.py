"""GPU parity of the re-quantizing epilogue (results written back as DyBit codes, Section III-B.1).

Oracle = the oracle's own GEMM / conv, then (ReLU), then the oracle's quantize with the given output scale, then
its pack: no new arithmetic.  int8-container layers must match bit for bit.  For the floating containers the fp32
value carries an accumulation tolerance, so the codes are checked against the oracle's encoder applied to the
GPU's own fp32 output (which the GEMM tests pin separately)."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _quant(x, fmt):
    packed, scale = dy.dybit_quantize_pack_2d(x.to(DEV), fmt)
    sp = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    return packed, scale, orc.quantize(x.numpy(), fmt[0], bool(fmt[1]), sp[1]), sp


def _expect(y_ref, fq, inv_q, relu):
    y = np.maximum(y_ref, 0) if relu else y_ref
    codes = orc.quantize(y.astype(np.float32), fq[0], bool(fq[1]), inv_q)
    return np.stack([orc.pack(r, fq[0])[: y.shape[1] * fq[0] // 8] for r in codes])


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (300, 520, 400), (777, 64, 1153), (64, 1000, 512), (5, 8, 77),
                                   (200, 264, 3100)])
@pytest.mark.parametrize("fq,relu", [((4, 0), True), ((4, 1), False), ((8, 1), False), ((2, 0), True), ((3, 1), False),
                                     ((6, 0), True)])
def test_gemm_requant_int8_container_bit_exact(M, N, K, fq, relu):
    fa, fb = (4, 0), (4, 1)
    a = wl.half_normal((M, K), seed=M + K)
    b = wl.normal((N, K), seed=N + K, std=0.05)
    pa, sa, ca, spa = _quant(a, fa)
    pb, sb, cb, spb = _quant(b, fb)
    _, y_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    # a "calibrated" output scale: slightly below the observed maximum, so that saturation is exercised too
    sq = orc.absmax_scale(y_ref * 0.9, fq[0], bool(fq[1]))
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    Q = dy.dybit_gemm_requant(M, N, K, pa, fa, sa, pb, fb, sb, fq, scale_q, relu=relu)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    assert np.array_equal(Q.cpu().numpy(), _expect(y_ref, fq, sq[1], relu))


def test_gemm_requant_padded_rows_feed_the_next_gemm():
    # layer 1 writes codes with GEMM-operand row padding; layer 2 consumes them directly
    fa, fb, fq = (4, 0), (4, 1), (4, 0)
    M, N1, K1, N2 = 200, 256, 300, 96
    a = wl.half_normal((M, K1), seed=1)
    w1 = wl.normal((N1, K1), seed=2, std=0.05)
    w2 = wl.normal((N2, N1), seed=3, std=0.05)
    pa, sa, ca, spa = _quant(a, fa)
    p1, s1, c1, sp1 = _quant(w1, fb)
    p2, s2, c2, sp2 = _quant(w2, fb)
    _, y1 = orc.gemm(ca, fa, spa[0], c1, fb, sp1[0])
    sq = orc.absmax_scale(np.maximum(y1, 0), fq[0], False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    ldq = dy.dybit_row_stride_bytes(N1, fq[0])
    Q = dy.dybit_gemm_requant(M, N1, K1, pa, fa, sa, p1, fb, s1, fq, scale_q, relu=True, ldq_bytes=ldq)
    C2, C2_raw = dy.dybit_gemm(M, N2, N1, Q, fq, scale_q, p2, fb, s2, want_raw=True)
    q_codes = orc.quantize(np.maximum(y1, 0), fq[0], False, sq[1])
    assert np.array_equal(Q.cpu().numpy(), orc.pack_rows(q_codes, fq[0]))
    S2, y2 = orc.gemm(q_codes, fq, sq[0], c2, fb, sp2[0])
    assert np.array_equal(C2_raw.cpu().numpy().astype(np.int64), S2)
    assert np.array_equal(C2.cpu().numpy(), y2)


@pytest.mark.parametrize("fa,fb", [((8, 0), (8, 1)), ((5, 0), (4, 1))])
def test_gemm_requant_float_containers_encode_their_own_output(fa, fb):
    M, N, K, fq = 260, 320, 500, (4, 0)
    a = wl.half_normal((M, K), seed=4)
    b = wl.normal((N, K), seed=5, std=0.05)
    pa, sa, _, _ = _quant(a, fa)
    pb, sb, _, _ = _quant(b, fb)
    C, _ = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb)
    y_gpu = C.cpu().numpy()
    sq = orc.absmax_scale(np.maximum(y_gpu, 0), fq[0], False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    Q = dy.dybit_gemm_requant(M, N, K, pa, fa, sa, pb, fb, sb, fq, scale_q, relu=True)
    assert np.array_equal(Q.cpu().numpy(), _expect(y_gpu, fq, sq[1], True))


@pytest.mark.parametrize("layer", [
    wl.ConvLayer("c64_3x3", 4, 28, 28, 64, 64, 3, 3, 1, 1),
    wl.ConvLayer("c128_3x3_s2", 4, 20, 20, 128, 96, 3, 3, 2, 1),
    wl.ConvLayer("stem_c3_7x7", 2, 32, 32, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("pointwise", 3, 14, 14, 256, 128, 1, 1, 1, 0),
    wl.ConvLayer("small_gather", 2, 8, 8, 64, 40, 3, 3, 1, 1),
], ids=lambda L: L.name)
def test_conv_requant_chains_into_the_next_conv(layer):
    fx, fw, fq = (4, 0), (4, 1), (4, 0)
    L = layer
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=7)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=8)
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    spx = orc.absmax_scale(x.numpy(), 4, False)
    spw = orc.absmax_scale(w.numpy(), 4, True)
    cx = orc.quantize(x.numpy(), 4, False, spx[1])
    cw = orc.quantize(w.numpy(), 4, True, spw[1])
    _, y = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=L.stride, pad=L.pad)
    sq = orc.absmax_scale(np.maximum(y, 0) * 0.95, 4, False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Q = dy.dybit_conv2d_requant(desc, px, fx, sx, pw, fw, sw, fq, scale_q, relu=True)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    q_codes = orc.quantize(np.maximum(y, 0), 4, False, sq[1])
    assert np.array_equal(Q.cpu().numpy(), orc.pack(q_codes, 4))
    # the stream is the next layer's X: a 1x1 conv on it must match the oracle on the oracle's codes
    k2 = 32
    w2 = wl.kaiming_normal(k2, 1, 1, L.k, seed=9)
    pw2, sw2 = dy.dybit_quantize_pack_2d(w2.reshape(k2, -1).to(DEV), fw)
    spw2 = orc.absmax_scale(w2.numpy(), 4, True)
    cw2 = orc.quantize(w2.numpy(), 4, True, spw2[1])
    d2 = dy.ConvDesc(L.n, L.oh, L.ow, L.k, k2, 1, 1, 1, 0, 1)
    Y2, Y2_raw = dy.dybit_conv2d(d2, Q, fq, scale_q, pw2, fw, sw2, want_raw=True)
    S2, y2 = orc.conv2d(q_codes, fq, sq[0], cw2, fw, spw2[0])
    assert np.array_equal(Y2_raw.cpu().numpy().astype(np.int64), S2)
    assert np.array_equal(Y2.cpu().numpy(), y2)


@pytest.mark.parametrize("M,N,K,fq,relu", [(300, 520, 400, (4, 0), True), (130, 72, 1153, (4, 1), False),
                                          (64, 1000, 512, (8, 1), False), (200, 264, 200, (3, 0), True)])
def test_gemm_requant_bias_is_added_in_fp32_before_relu(M, N, K, fq, relu):
    fa, fb = (4, 0), (4, 1)
    a = wl.half_normal((M, K), seed=M + K)
    b = wl.normal((N, K), seed=N + K, std=0.05)
    pa, sa, ca, spa = _quant(a, fa)
    pb, sb, cb, spb = _quant(b, fb)
    _, y_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    # biases of the size of the outputs, both signs, so that they flip codes and the ReLU decision
    bias = (wl.normal((N,), seed=N, std=float(np.abs(y_ref).mean()))).numpy().astype(np.float32)
    y_b = (y_ref.astype(np.float32) + bias[None, :]).astype(np.float32)
    sq = orc.absmax_scale(y_b * 0.9, fq[0], bool(fq[1]))
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    Q = dy.dybit_gemm_requant(M, N, K, pa, fa, sa, pb, fb, sb, fq, scale_q, relu=relu,
                              bias=torch.from_numpy(bias).to(DEV))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    assert np.array_equal(Q.cpu().numpy(), _expect(y_b, fq, sq[1], relu))
    # and the bias does change the result
    Q0 = dy.dybit_gemm_requant(M, N, K, pa, fa, sa, pb, fb, sb, fq, scale_q, relu=relu)
    assert not np.array_equal(Q.cpu().numpy(), Q0.cpu().numpy())


def test_conv_requant_bias_per_output_channel():
    fx, fw, fq = (4, 0), (4, 1), (4, 0)
    L = wl.ConvLayer("c64_3x3", 4, 28, 28, 64, 72, 3, 3, 1, 1)
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=17)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=18)
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    spx = orc.absmax_scale(x.numpy(), 4, False)
    spw = orc.absmax_scale(w.numpy(), 4, True)
    cx = orc.quantize(x.numpy(), 4, False, spx[1])
    cw = orc.quantize(w.numpy(), 4, True, spw[1])
    _, y = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=L.stride, pad=L.pad)
    bias = wl.normal((L.k,), seed=19, std=float(np.abs(y).mean())).numpy().astype(np.float32)
    y_b = (y.astype(np.float32) + bias.reshape(1, 1, 1, -1)).astype(np.float32)
    sq = orc.absmax_scale(np.maximum(y_b, 0) * 0.95, 4, False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Q = dy.dybit_conv2d_requant(desc, px, fx, sx, pw, fw, sw, fq, scale_q, relu=True,
                                bias=torch.from_numpy(bias).to(DEV))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    q_codes = orc.quantize(np.maximum(y_b, 0), 4, False, sq[1])
    assert np.array_equal(Q.cpu().numpy(), orc.pack(q_codes, 4))


def test_requant_argument_errors():
    one = torch.tensor([1.0, 1.0], device=DEV)
    pa = torch.zeros((4, 64), dtype=torch.uint8, device=DEV)
    with pytest.raises(dy.DybitError) as e:       # N * bits not a whole number of bytes
        dy.dybit_gemm_requant(4, 3, 128, pa, (4, 1), one, pa, (4, 1), one, (3, 0), one, Q=torch.zeros((4, 4), dtype=torch.uint8, device=DEV), ldq_bytes=4)
    assert e.value.status == 1
    with pytest.raises(dy.DybitError) as e:       # rows shorter than N codes
        dy.dybit_gemm_requant(4, 4, 128, pa, (4, 1), one, pa, (4, 1), one, (8, 0), one, Q=torch.zeros((4, 4), dtype=torch.uint8, device=DEV), ldq_bytes=0)
    assert e.value.status == 1


# the whole layer in one call: fp32 activation -> codes -> conv -> bias + ReLU -> packed output codes
@pytest.mark.parametrize("layer", [
    wl.ConvLayer("c64_3x3_im2col", 4, 28, 28, 64, 72, 3, 3, 1, 1),
    wl.ConvLayer("c3_7x7_stem", 2, 40, 40, 3, 64, 7, 7, 2, 3),
    wl.ConvLayer("c256_1x1", 3, 14, 14, 256, 128, 1, 1, 1, 0),
    wl.ConvLayer("c20_patch", 2, 9, 11, 20, 24, 3, 3, 1, 1),
], ids=lambda L: L.name)
def test_quantize_conv_requant_one_call(layer):
    fx, fw, fq = (4, 0), (4, 1), (4, 0)
    L = layer
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=31)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=32)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    spx = orc.absmax_scale(x.numpy(), 4, False)
    spw = orc.absmax_scale(w.numpy(), 4, True)
    cx = orc.quantize(x.numpy(), 4, False, spx[1])
    cw = orc.quantize(w.numpy(), 4, True, spw[1])
    _, y = orc.conv2d(cx, fx, spx[0], cw, fw, spw[0], stride=L.stride, pad=L.pad)
    bias = wl.normal((L.k,), seed=33, std=float(np.abs(y).mean())).numpy().astype(np.float32)
    y_b = (y.astype(np.float32) + bias.reshape(1, 1, 1, -1)).astype(np.float32)
    sq = orc.absmax_scale(np.maximum(y_b, 0) * 0.9, 4, False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Q, packed, scale = dy.dybit_quantize_conv2d_requant(desc, x.to(DEV), fx, pw, fw, sw, fq, scale_q, relu=True,
                                                        bias=torch.from_numpy(bias).to(DEV))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    assert scale.cpu().numpy().tolist() == [float(np.float32(spx[0])), float(np.float32(spx[1]))]
    assert np.array_equal(packed.cpu().numpy(), orc.pack(cx, 4))
    assert np.array_equal(Q.cpu().numpy(), orc.pack(orc.quantize(np.maximum(y_b, 0), 4, False, sq[1]), 4))
    # and the same bits as the two-call path
    px, sx = dy.dybit_quantize_pack(x.to(DEV), fx)
    Q2 = dy.dybit_conv2d_requant(desc, px, fx, sx, pw, fw, sw, fq, scale_q, relu=True, bias=torch.from_numpy(bias).to(DEV))
    assert torch.equal(Q, Q2)


# the same epilogue on layers that went through the folded launches (dybit_quantize_expand_layers, then
# dybit_conv2d_prepared with Q set): one layer leaves as codes with bias + ReLU, one as codes without, one as fp32
def test_layers_with_the_requant_epilogue():
    fx, fw, fq = (4, 0), (4, 1), (4, 0)
    shapes = [wl.ConvLayer("c64_3x3", 4, 28, 28, 64, 64, 3, 3, 1, 1), wl.ConvLayer("c128_1x1", 3, 14, 14, 128, 256, 1, 1, 1, 0),
              wl.ConvLayer("c3_stem", 2, 32, 32, 3, 64, 7, 7, 2, 3)]
    args, expect = [], []
    for i, L in enumerate(shapes):
        x = wl.half_normal((L.n, L.h, L.w, L.c), seed=41 + i)
        w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=51 + i)
        pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
        spx = orc.absmax_scale(x.numpy(), 4, False)
        spw = orc.absmax_scale(w.numpy(), 4, True)
        _, y = orc.conv2d(orc.quantize(x.numpy(), 4, False, spx[1]), fx, spx[0], orc.quantize(w.numpy(), 4, True, spw[1]), fw,
                          spw[0], stride=L.stride, pad=L.pad)
        a = dict(desc=dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1), X=x.to(DEV), fx=fx, W=pw, fw=fw,
                 scale_w=sw)
        if i == 0:
            bias = wl.normal((L.k,), seed=61, std=float(np.abs(y).mean())).numpy().astype(np.float32)
            y = np.maximum((y.astype(np.float32) + bias.reshape(1, 1, 1, -1)).astype(np.float32), 0)
            a.update(bias=torch.from_numpy(bias).to(DEV), relu=True)
        if i < 2:
            sq = orc.absmax_scale(np.abs(y) * 0.9, 4, False)
            a.update(fq=fq, scale_q=torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV))
            expect.append(orc.pack(orc.quantize(y if i == 0 else y.astype(np.float32), 4, False, sq[1]), 4))
        else:
            expect.append(y)
        args.append(a)
    layers = dy.ConvLayers(args)
    dy.dybit_quantize_expand_layers(layers)
    outs = [dy.dybit_conv2d_prepared(layers, i)[0] for i in range(len(shapes))]
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    for i, L in enumerate(shapes):
        assert np.array_equal(outs[i].cpu().numpy(), expect[i]), L.name
    # shared launches give the same codes and outputs
    for o in outs:
        o.zero_()
    dy.dybit_conv2d_prepared_layers(layers)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    for i, L in enumerate(shapes):
        assert np.array_equal((layers.Q[i] if layers.Q[i] is not None else layers.Y[i]).cpu().numpy(), expect[i]), L.name
    # and bit for bit the one-layer call
    a = args[0]
    Q1, _, _ = dy.dybit_quantize_conv2d_requant(a["desc"], a["X"], fx, a["W"], fw, a["scale_w"], fq, a["scale_q"], relu=True,
                                                bias=a["bias"])
    assert torch.equal(Q1, outs[0])


# products large enough for the CTA-pair kernel: its epilogue re-quantizes too (bias, ReLU, ragged last tiles)
@pytest.mark.parametrize("M,N,K,fq,relu,with_bias", [(2304, 2304, 256, (4, 0), True, False),
                                                      (2400, 2344, 200, (8, 1), False, True),
                                                      (2404, 2312, 130, (2, 0), True, True)])
def test_gemm_requant_on_cta_pairs(M, N, K, fq, relu, with_bias):
    fa, fb = (4, 0), (4, 1)
    a = wl.half_normal((M, K), seed=M + K)
    b = wl.normal((N, K), seed=N + K, std=0.05)
    pa, sa, ca, spa = _quant(a, fa)
    pb, sb, cb, spb = _quant(b, fb)
    _, y_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    bias = None
    if with_bias:
        bias = wl.normal((N,), seed=7, std=float(np.abs(y_ref).mean())).numpy().astype(np.float32)
        y_ref = (y_ref.astype(np.float32) + bias.reshape(1, -1)).astype(np.float32)
    sq = orc.absmax_scale(y_ref * 0.9, fq[0], bool(fq[1]))
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    Q = dy.dybit_gemm_requant(M, N, K, pa, fa, sa, pb, fb, sb, fq, scale_q, relu=relu,
                              bias=None if bias is None else torch.from_numpy(bias).to(DEV))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    assert np.array_equal(Q.cpu().numpy(), _expect(y_ref, fq, sq[1], relu))
