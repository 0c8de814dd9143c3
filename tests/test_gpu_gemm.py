"""GPU parity: dybit_gemm against the CPU oracle.

int8 container (both formats with <= 4 magnitude bits): raw int32 sums and
fp32 outputs must be bit-exact.  fp8 / bf16 containers accumulate in fp32:
|err| <= 1e-5 * K * max|a| * max|b| with a, b the dequantised operands.
"""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def quantize_operand(x: torch.Tensor, fmt):
    """x [rows][K] fp32 on host -> (packed dev tensor, scale dev tensor, oracle codes, oracle scale)."""
    packed, scale = dy.dybit_quantize_pack_2d(x.to(DEV), fmt)
    sp = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    codes = orc.quantize(x.numpy(), fmt[0], bool(fmt[1]), sp[1])
    return packed, scale, codes, sp


def check_gemm(M, N, K, fa, fb, seed=0, a_dist=None, b_std=1.0):
    a = (a_dist or wl.normal)((M, K), seed=seed)
    if not fa[1]:
        a = a.abs()
    b = wl.normal((N, K), seed=seed + 1, std=b_std)
    if not fb[1]:
        b = b.abs()
    pa, sa, ca, spa = quantize_operand(a, fa)
    pb, sb, cb, spb = quantize_operand(b, fb)
    # the packed operands themselves are already covered by the quantize tests; assert anyway
    assert np.array_equal(pa.cpu().numpy(), orc.pack_rows(ca, fa[0]))
    assert np.array_equal(pb.cpu().numpy(), orc.pack_rows(cb, fb[0]))
    cont, _, _ = dy.dybit_choose_container(fa, fb)
    C, C_raw = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb, want_raw=(cont == 0))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    S, C_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    if cont == 0:
        assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S)
        assert np.array_equal(C.cpu().numpy(), C_ref)
    else:
        amax = float(spa[0]) * float(np.abs(orc.decode_table(fa[0], bool(fa[1]))).max())
        bmax = float(spb[0]) * float(np.abs(orc.decode_table(fb[0], bool(fb[1]))).max())
        tol = 1e-5 * K * amax * bmax
        err = np.abs(C.cpu().numpy().astype(np.float64) - C_ref.astype(np.float64)).max()
        assert err <= tol, (err, tol)
    return cont


def test_config1_tiny_4bit():
    # W 256x256 ~ N(0, 0.02), X 64x256 half-normal, 4-bit both, X * W^T
    x = wl.half_normal((64, 256), seed=0)
    w = wl.normal((256, 256), seed=0, std=0.02)
    for fx in ((4, 0), (4, 1)):
        px, sx, cx, spx = quantize_operand(x, fx)
        pw, sw, cw, spw = quantize_operand(w, (4, 1))
        C, C_raw = dy.dybit_gemm(64, 256, 256, px, fx, sx, pw, (4, 1), sw, want_raw=True)
        S, C_ref = orc.gemm(cx, fx, spx[0], cw, (4, 1), spw[0])
        assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S)
        assert np.array_equal(C.cpu().numpy(), C_ref)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (128, 256, 128), (129, 257, 129), (300, 520, 400),
                                   (64, 1000, 512), (777, 64, 1153), (1000, 130, 77), (256, 256, 2048)])
def test_int8_container_bit_exact(M, N, K):
    assert check_gemm(M, N, K, (4, 1), (4, 1), seed=M + N + K) == 0


@pytest.mark.parametrize("fa,fb", [((2, 1), (2, 1)), ((3, 1), (4, 0)), ((5, 1), (3, 0)), ((4, 0), (2, 1)),
                                   ((3, 0), (5, 1))])
def test_int8_container_all_narrow_formats(fa, fb):
    assert check_gemm(200, 300, 333, fa, fb, seed=fa[0] * 8 + fb[0]) == 0


@pytest.mark.parametrize("fa,fb", [((5, 0), (4, 1)), ((6, 1), (6, 1)), ((5, 0), (6, 1)), ((2, 1), (5, 0))])
def test_e4m3_container_within_tolerance(fa, fb):
    assert check_gemm(260, 300, 700, fa, fb, seed=fa[0] * 8 + fb[0]) == 1


@pytest.mark.parametrize("fa,fb", [((8, 1), (8, 1)), ((8, 0), (4, 1)), ((6, 0), (7, 1)), ((7, 0), (2, 1)),
                                   ((6, 0), (5, 0))])
def test_bf16_container_within_tolerance(fa, fb):
    assert check_gemm(260, 300, 700, fa, fb, seed=fa[0] * 8 + fb[0]) == 2


# Few output tiles and a long K (many K blocks per tile, several trips round the stage ring, narrowed tiles):
# every container, ragged M / N / K.  (The library does not split K: each tile's contraction runs in one CTA.)
@pytest.mark.parametrize("M,N,K,fa,fb,cont", [
    (130, 70, 1100, (4, 1), (4, 1), 0),
    (64, 1000, 4096, (4, 0), (4, 1), 0),
    (257, 300, 5003, (3, 1), (5, 1), 0),
    (1, 1, 3000, (2, 1), (4, 0), 0),
    (700, 129, 2500, (4, 1), (2, 1), 0),
    (260, 300, 3000, (5, 0), (4, 1), 1),
    (100, 520, 1500, (8, 1), (8, 1), 2),
    (500, 64, 2111, (6, 0), (7, 1), 2),
])
def test_few_tiles_long_k(M, N, K, fa, fb, cont):
    assert check_gemm(M, N, K, fa, fb, seed=M + N + K) == cont


def test_same_shape_three_times_in_a_row():
    for seed in (1, 2, 3):
        assert check_gemm(256, 256, 2048, (4, 1), (4, 1), seed=seed) == 0


def test_many_tiles_persistent_schedule():
    # more tiles than SMs with ragged edges in every dimension: each CTA runs several tiles
    assert check_gemm(128 * 13 + 5, 256 * 12 + 9, 256 + 3, (4, 1), (4, 0), seed=7) == 0


def test_all_codes_every_product():
    # every pair of 4-bit signed codes meets at least once; K=1 rows
    fa = fb = (4, 1)
    a_codes = np.repeat(np.arange(16, dtype=np.uint8), 16)[:, None]
    b_codes = np.arange(16, dtype=np.uint8)[:, None]
    pa = torch.from_numpy(orc.pack_rows(a_codes, 4)).to(DEV)
    pb = torch.from_numpy(orc.pack_rows(b_codes, 4)).to(DEV)
    one = torch.tensor([1.0, 1.0], device=DEV)
    C, C_raw = dy.dybit_gemm(256, 16, 1, pa, fa, one, pb, fb, one, want_raw=True)
    S, C_ref = orc.gemm(a_codes, fa, 1.0, b_codes, fb, 1.0)
    assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S)
    assert np.array_equal(C.cpu().numpy(), C_ref)


def test_gemm_argument_errors():
    fa = fb = (4, 1)
    pa = torch.zeros((4, 64), dtype=torch.uint8, device=DEV)
    one = torch.tensor([1.0, 1.0], device=DEV)
    ws = torch.zeros(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(dy.DybitError) as e:
        dy.dybit_gemm(4, 4, 128, pa, fa, one, pa, fb, one, ws=torch.zeros(2048, dtype=torch.uint8, device=DEV))
    assert e.value.status == 4           # workspace too small
    with pytest.raises(dy.DybitError) as e:
        dy.dybit_gemm(4, 4, 256, pa, fa, one, pa, fb, one)
    assert e.value.status == 1           # row stride smaller than K needs
    with pytest.raises(dy.DybitError) as e:
        dy.dybit_gemm(4, 4, 128, pa, (8, 1), one, pa, (8, 1), one, want_raw=True, lda_bytes=128, ldb_bytes=128)
    assert e.value.status in (1, 2)
    del ws


def test_profile_clock_brackets_the_kernel():
    # the device-clock hook: start and end stamps of the tensor-core kernel, result unchanged
    fa = fb = (4, 1)
    M, N, K = 300, 200, 384
    a = wl.normal((M, K), seed=11)
    b = wl.normal((N, K), seed=12)
    pa, sa = dy.dybit_quantize_pack_2d(a.to(DEV), fa)
    pb, sb = dy.dybit_quantize_pack_2d(b.to(DEV), fb)
    C0, _ = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb)
    t2 = torch.tensor([-1, 0], dtype=torch.int64, device=DEV)
    dy.dybit_profile_next_gemm_clock(t2)
    C1, _ = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb)
    torch.cuda.synchronize()
    start, end = t2.cpu().tolist()
    assert start > 0 and end > start and end - start < 10_000_000        # nanoseconds
    assert torch.equal(C0, C1)
    # disarmed after one kernel: the pair stays as it is
    before = t2.clone()
    dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb)
    torch.cuda.synchronize()
    assert torch.equal(before, t2)


# Large products run on CTA pairs (256 x 256 tiles, cta_group::2), with or without raw sums; both calls must give
# the oracle's results.  On 74 pairs the 81-100 tiles of the first cases leave a last wave that is less than half full,
# which the kernel works on as 256 x 128 halves (in "half_empty_pair" the right half of the last column of tiles is
# empty); the 121 tiles of the last case leave 47, which stay whole.
@pytest.mark.parametrize("M,N,K,fa,fb", [
    (2304, 2304, 256, (4, 1), (4, 1)),        # whole tiles
    (2500, 2400, 384, (4, 1), (4, 0)),        # ragged in M (196 rows in the last block: both CTAs of the pair have rows) and N
    (2404, 2308, 130, (3, 1), (4, 1)),        # last block has 100 rows: the pair's second CTA has none
    (2304, 2304, 200, (5, 1), (5, 0)),        # e4m3 container
    (2304, 2560, 136, (8, 1), (6, 0)),        # bf16 container
    (2816, 2700, 160, (4, 1), (4, 0)),        # 121 tiles: no halves
], ids=["whole", "ragged", "half_empty_pair", "e4m3", "bf16", "last_wave_whole"])
def test_cta_pair_kernel(M, N, K, fa, fb):
    a = wl.normal((M, K), seed=M + K)
    if not fa[1]:
        a = a.abs()
    b = wl.normal((N, K), seed=N + K)
    if not fb[1]:
        b = b.abs()
    pa, sa, ca, spa = quantize_operand(a, fa)
    pb, sb, cb, spb = quantize_operand(b, fb)
    cont, _, _ = dy.dybit_choose_container(fa, fb)
    C, _ = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    S, C_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    if cont == 0:
        assert np.array_equal(C.cpu().numpy(), C_ref)
        C1, C_raw = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb, want_raw=True)
        assert torch.equal(C, C1)
        assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S)
    else:
        amax = float(spa[0]) * float(np.abs(orc.decode_table(fa[0], bool(fa[1]))).max())
        bmax = float(spb[0]) * float(np.abs(orc.decode_table(fb[0], bool(fb[1]))).max())
        err = np.abs(C.cpu().numpy().astype(np.float64) - C_ref.astype(np.float64)).max()
        assert err <= 1e-5 * K * amax * bmax, err


# The B operand decoded in the GEMM's main loop (packed 4-bit weights -> int8 through the register table, written into
# the swizzled operand tile by decode warps) instead of expanded by a separate launch: forced on for every shape here
# (by default only few-row products take it), and compared with the oracle AND with the expand path, bit for bit.
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (32, 1000, 512), (128, 256, 128), (129, 257, 129), (300, 520, 400),
                                   (7, 4100, 2000), (256, 64, 4096), (1000, 130, 77), (513, 768, 1153)])
@pytest.mark.parametrize("fa,fb", [((4, 0), (4, 1)), ((4, 1), (4, 0)), ((2, 1), (4, 1)), ((5, 1), (4, 1))])
def test_weights_decoded_in_the_main_loop(M, N, K, fa, fb):
    a = wl.normal((M, K), seed=M + K)
    if not fa[1]:
        a = a.abs()
    b = wl.normal((N, K), seed=N + K + 1, std=0.3)
    if not fb[1]:
        b = b.abs()
    pa, sa, ca, spa = quantize_operand(a, fa)
    pb, sb, cb, spb = quantize_operand(b, fb)
    S, C_ref = orc.gemm(ca, fa, spa[0], cb, fb, spb[0])
    outs = []
    try:
        for mode in (1, 0):
            dy.dybit_set_gemm_decode(mode)
            launches = dy.dybit_launch_count()
            C, C_raw = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb, want_raw=True)
            torch.cuda.synchronize()
            assert dy.dybit_last_device_status() == (0, 0)
            # the tensor-core kernel + one expand launch (two when A and B need different expand kernels)
            assert dy.dybit_launch_count() - launches <= 3
            assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S), mode
            assert np.array_equal(C.cpu().numpy(), C_ref), mode
            outs.append(C)
    finally:
        dy.dybit_set_gemm_decode(2)
    assert torch.equal(outs[0], outs[1])


def test_gemm_decode_mode_argument():
    with pytest.raises(dy.DybitError):
        dy.dybit_set_gemm_decode(5)
    dy.dybit_set_gemm_decode(2)
