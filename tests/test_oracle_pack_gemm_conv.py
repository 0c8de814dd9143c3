"""Pins for the oracle's packing, GEMM and convolution.

Packing is pinned to numpy's bit routines, GEMM to numpy's integer / fp64
matrix product on separately decoded operands, convolution to torch's fp64
conv2d; plus tiny brute-force cases, identities and checksums that hold at
any size.
"""
import numpy as np
import pytest
import torch

from oracle import dybit_oracle as orc

FORMATS = [(b, s) for b in range(2, 9) for s in (False, True)]


def _m(fmt):
    return fmt[0] - 1 if fmt[1] else fmt[0]


def _ints(codes, fmt):
    """Integer images via the (separately pinned) decode table."""
    tab = orc.decode_table(*fmt) * 2.0 ** (_m(fmt) - 1)
    assert np.all(tab == np.round(tab))
    return tab.astype(np.int64)[codes]


# ------------------------------------------------------------------ packing

@pytest.mark.parametrize("bits", range(2, 9))
def test_pack_is_a_little_endian_bit_stream(bits):
    rng = np.random.default_rng(bits)
    for n in (0, 1, 7, 128, 1000, 4099):
        codes = rng.integers(0, 1 << bits, n, dtype=np.uint8)
        packed = orc.pack(codes, bits)
        assert packed.size == orc.packed_bytes(n, bits) and packed.size % 16 == 0
        # numpy: bit b of code j, LSB first, concatenated, 8 per byte LSB first
        bitmat = np.unpackbits(codes[:, None], axis=1, bitorder="little")[:, :bits]
        want = np.packbits(bitmat.ravel(), bitorder="little")
        assert np.array_equal(packed[:want.size], want)
        assert not packed[want.size:].any()
        assert np.array_equal(orc.unpack(packed, n, bits), codes)


@pytest.mark.parametrize("bits", range(2, 9))
def test_pack_rows_pads_each_row_with_code_zero(bits):
    rng = np.random.default_rng(bits + 50)
    rows, cols = 5, 300
    codes = rng.integers(0, 1 << bits, (rows, cols), dtype=np.uint8)
    rs = orc.row_stride_bytes(cols, bits)
    assert rs == 384 * bits // 8 and rs % 16 == 0
    packed = orc.pack_rows(codes, bits)
    assert packed.shape == (rows, rs)
    for r in range(rows):
        assert np.array_equal(packed[r], np.pad(orc.pack(codes[r], bits), (0, rs))[:rs])
        assert np.array_equal(orc.unpack(packed[r], 384, bits)[cols:], np.zeros(84, np.uint8))
    assert np.array_equal(orc.unpack_rows(packed, rows, cols, bits), codes)


def test_all_codes_round_trip():
    for bits in range(2, 9):
        codes = np.arange(1 << bits, dtype=np.uint8)
        assert np.array_equal(orc.unpack(orc.pack(codes, bits), codes.size, bits), codes)


def test_dequantize_is_scale_times_value():
    for fmt in FORMATS:
        codes = np.arange(1 << fmt[0], dtype=np.uint8)
        got = orc.dequantize(codes, fmt[0], fmt[1], 0.3)
        want = (np.float32(0.3) * orc.decode_table(*fmt).astype(np.float32)).astype(np.float32)
        assert np.array_equal(got, want)


# --------------------------------------------------------------------- GEMM

@pytest.mark.parametrize("fa,fb", [((4, True), (4, False)), ((8, True), (8, True)),
                                   ((2, True), (6, False)), ((5, False), (3, True)),
                                   ((8, False), (4, True))])
def test_gemm_against_numpy(fa, fb):
    rng = np.random.default_rng(fa[0] * 10 + fb[0])
    M, N, K = 9, 13, 157
    A = rng.integers(0, 1 << fa[0], (M, K), dtype=np.uint8)
    B = rng.integers(0, 1 << fb[0], (N, K), dtype=np.uint8)
    sa, sb = np.float32(0.0123), np.float32(1.75)
    S, C = orc.gemm(A, fa, sa, B, fb, sb)
    S_np = _ints(A, fa) @ _ints(B, fb).T                      # exact int64
    assert np.array_equal(S, S_np)
    # real-valued definition in fp64 on dequantised operands
    real = (float(sa) * orc.decode_table(*fa)[A]) @ (float(sb) * orc.decode_table(*fb)[B]).T
    assert np.allclose(C, real, rtol=3e-7, atol=0)
    # the stated final arithmetic: one int->fp32 conversion, one fp32 multiply
    al = np.float32(float(sa) * float(sb) * 2.0 ** -((_m(fa) - 1) + (_m(fb) - 1)))
    assert orc.alpha(sa, fa, sb, fb) == al
    assert np.array_equal(C, S.astype(np.float32) * al)


def test_gemm_tiny_brute_force():
    fa, fb = (4, True), (4, False)
    ta, tb = orc.decode_table(*fa), orc.decode_table(*fb)
    for a in range(16):
        for b in range(16):
            S, C = orc.gemm(np.array([[a]], np.uint8), fa, 1.0, np.array([[b]], np.uint8), fb, 1.0)
            assert C[0, 0] == np.float32(ta[a] * tb[b])
            assert S[0, 0] == int(ta[a] * 4) * int(tb[b] * 8)
    # two-term dot product, operands transposed on purpose: C = A * B^T, not A^T * B
    A = np.array([[1, 2], [3, 4]], np.uint8)           # 0.125 .25 / .375 .5
    B = np.array([[8, 0], [0, 12]], np.uint8)          # 1 0 / 0 2
    _, C = orc.gemm(A, (4, False), 1.0, B, (4, False), 1.0)
    assert np.array_equal(C, np.array([[0.125, 0.5], [0.375, 1.0]], np.float32))


def test_gemm_one_hot_operand_reproduces_the_other():
    fa, fb = (4, False), (5, True)
    K = 40
    one = 8                                            # Table I: pattern 1000 is 1.0
    A = np.zeros((K, K), np.uint8)
    A[np.arange(K), np.arange(K)] = one
    rng = np.random.default_rng(1)
    B = rng.integers(0, 32, (7, K), dtype=np.uint8)
    _, C = orc.gemm(A, fa, 1.0, B, fb, 1.0)
    assert np.array_equal(C, orc.decode_table(*fb)[B].T.astype(np.float32))


def test_gemm_checksums_and_sampling():
    fa, fb = (4, True), (4, True)
    rng = np.random.default_rng(2)
    M, N, K = 31, 17, 300
    A = rng.integers(0, 16, (M, K), dtype=np.uint8)
    B = rng.integers(0, 16, (N, K), dtype=np.uint8)
    S, C = orc.gemm(A, fa, 0.5, B, fb, 0.25)
    IA, IB = _ints(A, fa), _ints(B, fb)
    assert np.array_equal(S.sum(axis=0), IA.sum(axis=0) @ IB.T)
    assert np.array_equal(S.sum(axis=1), IA @ IB.sum(axis=0))
    ri = rng.integers(0, M, 50)
    ci = rng.integers(0, N, 50)
    Ss, Cs = orc.gemm_sampled(A, fa, 0.5, B, fb, 0.25, ri, ci)
    assert np.array_equal(Ss, S[ri, ci]) and np.array_equal(Cs, C[ri, ci])


def test_gemm_ignores_row_padding():
    # codes appended as 0 contribute exactly nothing
    fa = fb = (3, True)
    rng = np.random.default_rng(4)
    A = rng.integers(0, 8, (4, 50), dtype=np.uint8)
    B = rng.integers(0, 8, (6, 50), dtype=np.uint8)
    S0, _ = orc.gemm(A, fa, 1.0, B, fb, 1.0)
    S1, _ = orc.gemm(np.pad(A, ((0, 0), (0, 78))), fa, 1.0, np.pad(B, ((0, 0), (0, 78))), fb, 1.0)
    assert np.array_equal(S0, S1)


# --------------------------------------------------------------------- conv

@pytest.mark.parametrize("r,stride,pad,dil", [(3, 1, 1, 1), (3, 2, 1, 1), (1, 1, 0, 1),
                                              (1, 2, 0, 1), (7, 2, 3, 1), (3, 1, 2, 2)])
def test_conv_against_torch_fp64(r, stride, pad, dil):
    fx, fw = (4, False), (4, True)
    rng = np.random.default_rng(r * 7 + stride)
    n, h, w, c, k = 2, 11, 9, 5, 6
    X = rng.integers(0, 16, (n, h, w, c), dtype=np.uint8)
    W = rng.integers(0, 16, (k, r, r, c), dtype=np.uint8)
    sx, sw = np.float32(0.37), np.float32(0.011)
    S, Y = orc.conv2d(X, fx, sx, W, fw, sw, stride=stride, pad=pad, dilation=dil)
    xr = torch.from_numpy(orc.decode_table(*fx)[X]).permute(0, 3, 1, 2)          # NCHW fp64
    wr = torch.from_numpy(orc.decode_table(*fw)[W]).permute(0, 3, 1, 2)          # KCRS fp64
    ref = torch.nn.functional.conv2d(xr, wr, stride=stride, padding=pad, dilation=dil)
    ref = ref.permute(0, 2, 3, 1).numpy()
    assert S.shape == ref.shape
    assert np.array_equal(S, np.round(ref * 2.0 ** (3 + 2)).astype(np.int64))
    assert np.allclose(Y, ref * float(sx) * float(sw), rtol=3e-7, atol=0)


def test_pointwise_conv_is_a_gemm():
    fx, fw = (6, False), (2, True)
    rng = np.random.default_rng(9)
    n, h, w, c, k = 2, 4, 5, 24, 10
    X = rng.integers(0, 64, (n, h, w, c), dtype=np.uint8)
    W = rng.integers(0, 4, (k, 1, 1, c), dtype=np.uint8)
    S, Y = orc.conv2d(X, fx, 0.1, W, fw, 0.2)
    Sg, Cg = orc.gemm(X.reshape(-1, c), fx, 0.1, W.reshape(k, c), fw, 0.2)
    assert np.array_equal(S.reshape(-1, k), Sg) and np.array_equal(Y.reshape(-1, k), Cg)


def test_conv_equals_gemm_on_explicit_patches():
    fx, fw = (4, True), (4, True)
    rng = np.random.default_rng(10)
    n, h, w, c, k, r, stride, pad = 1, 6, 7, 3, 4, 3, 2, 1
    X = rng.integers(0, 16, (n, h, w, c), dtype=np.uint8)
    W = rng.integers(0, 16, (k, r, r, c), dtype=np.uint8)
    S, _ = orc.conv2d(X, fx, 1.0, W, fw, 1.0, stride=stride, pad=pad)
    oh, ow = orc.conv_out_hw(h, w, r, r, stride, pad)
    patches = np.zeros((n * oh * ow, r * r * c), np.uint8)      # code 0 where the tap is outside
    row = 0
    for i in range(oh):
        for j in range(ow):
            for a in range(r):
                for b in range(r):
                    ih, iw = i * stride - pad + a, j * stride - pad + b
                    if 0 <= ih < h and 0 <= iw < w:
                        patches[row, (a * r + b) * c:(a * r + b + 1) * c] = X[0, ih, iw]
            row += 1
    Sg, _ = orc.gemm(patches, fx, 1.0, W.reshape(k, -1), fw, 1.0)
    assert np.array_equal(S.reshape(-1, k), Sg)


def test_sampled_conv_is_the_full_conv_on_quantised_input():
    fx, fw = (4, False), (3, True)
    rng = np.random.default_rng(12)
    n, h, w, c, k, r, stride, pad = 2, 9, 8, 6, 5, 3, 2, 1
    x = np.abs(rng.normal(size=(n, h, w, c))).astype(np.float32)
    W = rng.integers(0, 8, (k, r, r, c), dtype=np.uint8)
    sp = orc.absmax_scale(x, *fx)
    S, Y = orc.conv2d(orc.quantize(x, fx[0], fx[1], sp[1]), fx, sp[0], W, fw, 0.3, stride=stride, pad=pad)
    idx = rng.permutation(S.size)[:97]
    Ss, Ys = orc.conv2d_sampled(x, fx, sp, W, fw, 0.3, idx, stride=stride, pad=pad)
    assert np.array_equal(Ss, S.ravel()[idx]) and np.array_equal(Ys, Y.ravel()[idx])
