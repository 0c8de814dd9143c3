"""GPU parity: absmax / quantize+pack / decode against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
FORMATS = [(b, s) for b in range(2, 9) for s in (0, 1)]
DEV = "cuda:0"


def _oracle_pack(x_np, fmt, scale_pair=None):
    bits, sg = fmt
    if scale_pair is None:
        scale_pair = orc.absmax_scale(x_np, bits, bool(sg))
    codes = orc.quantize(x_np.ravel(), bits, bool(sg), scale_pair[1])
    return orc.pack(codes, bits), codes, scale_pair


def _edge_values(m):
    """Every midpoint between adjacent values and its fp32 neighbours, both signs, plus specials."""
    vals = np.array([orc.decode_mag(m, c) for c in range(1 << m)], dtype=np.float64)
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    pts = np.concatenate([vals.astype(np.float32), mids, np.nextafter(mids, np.float32(0)),
                          np.nextafter(mids, np.float32(np.inf)),
                          np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-40, -1e-40, 3e38, 1e-30,
                                    vals[-1] * 1.0000001, vals[-1] * 2], dtype=np.float32)])
    return np.concatenate([pts, -pts]).astype(np.float32)


@pytest.mark.parametrize("fmt", FORMATS)
def test_quantize_every_midpoint_and_special(fmt):
    bits, sg = fmt
    m = bits - 1 if sg else bits
    x = _edge_values(m)
    for inv in (1.0, 0.8125, 1.37):
        xs = (x / np.float32(inv)).astype(np.float32)
        scale = torch.tensor([1.0 / inv, inv], dtype=torch.float32, device=DEV)
        packed, _ = dy.dybit_quantize_pack(torch.from_numpy(xs).to(DEV), fmt, scale=scale)
        want, _, _ = _oracle_pack(xs, fmt, (np.float32(1.0 / inv), np.float32(inv)))
        assert np.array_equal(packed.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("n", [1, 31, 1024, 5000, 262144 + 77])
def test_quantize_pack_with_max_abs_scale(fmt, n):
    dist = wl.half_normal if not fmt[1] else (wl.laplace if n % 2 else wl.normal)
    x = dist((n,), seed=n + fmt[0])
    xd = x.to(DEV)
    packed, scale = dy.dybit_quantize_pack(xd, fmt)
    want, _, sp = _oracle_pack(x.numpy(), fmt)
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert packed.numel() == dy.dybit_packed_bytes(n, fmt[0])
    assert np.array_equal(packed.cpu().numpy(), want)
    # absmax alone gives the same pair
    assert torch.equal(dy.dybit_absmax_scale(xd, fmt), scale)


def test_quantize_empty_zero_and_nonfinite():
    fmt = (4, 1)
    packed, scale = dy.dybit_quantize_pack(torch.zeros(0, device=DEV), fmt)
    assert packed.numel() == 0 and scale.tolist() == [1.0, 1.0]
    packed, scale = dy.dybit_quantize_pack(torch.zeros(300, device=DEV), fmt)
    assert scale.tolist() == [1.0, 1.0] and not packed.any()
    x = wl.normal((4096,), 3)
    x[5], x[6], x[7] = float("nan"), float("inf"), float("-inf")
    packed, scale = dy.dybit_quantize_pack(x.to(DEV), fmt)
    want, _, sp = _oracle_pack(x.numpy(), fmt)
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert np.array_equal(packed.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", [(8, 0), (8, 1), (4, 1), (2, 1)])
def test_quantize_tiny_tensor_whose_reciprocal_scale_overflows(fmt):
    # max |x| = 1e-38: 2^(m-1) / amax is +inf in fp32, so a zero element meets 0 * inf = NaN, which must still encode to 0
    x = np.array([0.0, 1e-38, -1e-38, 0.0, -0.0, 5e-39] * 50, dtype=np.float32)
    packed, scale = dy.dybit_quantize_pack(torch.from_numpy(x).to(DEV), fmt)
    want, _, sp = _oracle_pack(x, fmt)
    assert np.isinf(sp[1]) or fmt == (2, 1)
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert np.array_equal(packed.cpu().numpy(), want)
    # the same with a caller-given pair whose reciprocal is +inf
    given = torch.tensor([1e-39, float("inf")], dtype=torch.float32, device=DEV)
    packed, _ = dy.dybit_quantize_pack(torch.from_numpy(x).to(DEV), fmt, scale=given)
    want, _, _ = _oracle_pack(x, fmt, (np.float32(1e-39), np.float32(np.inf)))
    assert np.array_equal(packed.cpu().numpy(), want)


def test_quantize_unaligned_input_pointer():
    fmt = (5, 1)
    base = wl.normal((10001,), 8)
    x = base[1:]                                   # 4-byte aligned only
    xd = base.to(DEV)[1:]
    assert xd.data_ptr() % 16 == 4
    packed, scale = dy.dybit_quantize_pack(xd.contiguous() if not xd.is_contiguous() else xd, fmt)
    want, _, sp = _oracle_pack(x.numpy(), fmt)
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert np.array_equal(packed.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", [(2, 1), (3, 1), (4, 1), (4, 0), (5, 0), (6, 1), (7, 0), (8, 1)])
@pytest.mark.parametrize("rows,cols,ld", [(5, 300, 300), (3, 1153, 1200), (130, 128, 128), (2, 2304, 2304)])
def test_quantize_pack_2d_rows(fmt, rows, cols, ld):
    x = wl.normal((rows, ld), seed=rows + cols)
    if not fmt[1]:
        x = x.abs()
    xd = x.to(DEV)
    packed, scale = dy.dybit_quantize_pack_2d(xd, fmt, cols=cols)
    used = x[:, :cols].contiguous().numpy()
    sp = orc.absmax_scale(used, fmt[0], bool(fmt[1]))
    codes = orc.quantize(used, fmt[0], bool(fmt[1]), sp[1])
    want = orc.pack_rows(codes, fmt[0])
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert packed.shape == want.shape
    assert np.array_equal(packed.cpu().numpy(), want)


def test_quantize_pack_2d_wide_stride_is_zero_filled():
    fmt = (4, 1)
    x = wl.normal((4, 200), 1)
    stride = dy.dybit_row_stride_bytes(200, 4) + 64
    packed = torch.full((4, stride), 0xAB, dtype=torch.uint8, device=DEV)
    dy.dybit_quantize_pack_2d(x.to(DEV), fmt, packed=packed, row_stride_bytes=stride)
    sp = orc.absmax_scale(x.numpy(), 4, True)
    want = orc.pack_rows(orc.quantize(x.numpy(), 4, True, sp[1]), 4, row_stride=stride)
    assert np.array_equal(packed.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("n", [1, 1000, 40000 + 3])
def test_decode_matches_oracle(fmt, n):
    rng = np.random.default_rng(n + fmt[0])
    codes = rng.integers(0, 1 << fmt[0], n, dtype=np.uint8)
    packed = torch.from_numpy(orc.pack(codes, fmt[0])).to(DEV)
    scale = torch.tensor([0.0371, 1 / 0.0371], dtype=torch.float32, device=DEV)
    out = dy.dybit_decode(packed, n, fmt, scale)
    want = orc.dequantize(codes, fmt[0], bool(fmt[1]), np.float32(0.0371))
    assert np.array_equal(out.cpu().numpy(), want)
    out1 = dy.dybit_decode(packed, n, fmt, None)
    assert np.array_equal(out1.cpu().numpy(), orc.dequantize(codes, fmt[0], bool(fmt[1]), np.float32(1.0)))


def test_round_trip_quantize_decode_large():
    # several hundred chunks and a ragged tail; sampled element-by-element against the oracle
    n = (1 << 22) + 12345
    fmt = (4, 1)
    x = wl.normal((n,), 42, device=DEV)
    packed, scale = dy.dybit_quantize_pack(x, fmt)
    xh = x.cpu().numpy()
    sp = orc.absmax_scale(xh, 4, True)
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    want = orc.pack(orc.quantize(xh, 4, True, sp[1]), 4)
    assert np.array_equal(packed.cpu().numpy(), want)
    back = dy.dybit_decode(packed, n, fmt, scale).cpu().numpy()
    assert np.array_equal(back, orc.dequantize(orc.unpack(want, n, 4), 4, True, sp[0]))
