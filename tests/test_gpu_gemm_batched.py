"""GPU parity of the batched GEMM: every entry against the oracle's GEMM on that entry (the batch is a loop of
independent products by definition).  int8 container: bit-exact; fp8 / bf16 containers: 1e-5 * K * max|a| * max|b|."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _quant3(x, fmt):
    """x [batch][rows][K] fp32 -> packed [batch][rows][row bytes] on the device with ONE scale for the tensor."""
    b, r, k = x.shape
    packed, scale = dy.dybit_quantize_pack_2d(x.reshape(b * r, k).to(DEV), fmt)
    sp = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    codes = orc.quantize(x.numpy(), fmt[0], bool(fmt[1]), sp[1]).reshape(b, r, k)
    return packed.reshape(b, r, -1), scale, codes, sp


def check(batch, M, N, K, fa, fb, seed=0, strided=False):
    a = wl.normal((batch, M, K), seed=seed)
    bm = wl.normal((batch, N, K), seed=seed + 1)
    if not fa[1]:
        a = a.abs()
    if not fb[1]:
        bm = bm.abs()
    pa, sa, ca, spa = _quant3(a, fa)
    pb, sb, cb, spb = _quant3(bm, fb)
    C = None
    if strided:
        # entries of A twice as far apart as they need to be; C with padded rows and a gap between entries
        wide = torch.zeros((batch, 2 * M, pa.shape[2]), dtype=torch.uint8, device=DEV)
        wide[:, :M] = pa
        pa = wide[:, :M]
        buf = torch.full((batch, M + 3, N + 4), -7.0, dtype=torch.float32, device=DEV)
        C = buf[:, :M, :N]
    cont, _, _ = dy.dybit_choose_container(fa, fb)
    C, C_raw = dy.dybit_gemm_batched(M, N, K, pa, fa, sa, pb, fb, sb, want_raw=(cont == 0 and not strided), C=C)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    got = C.cpu().numpy()
    for i in range(batch):
        S, ref = orc.gemm(ca[i], fa, spa[0], cb[i], fb, spb[0])
        if cont == 0:
            assert np.array_equal(got[i], ref), i
            if C_raw is not None:
                assert np.array_equal(C_raw[i].cpu().numpy().astype(np.int64), S), i
        else:
            amax = float(spa[0]) * float(np.abs(orc.decode_table(fa[0], bool(fa[1]))).max())
            bmax = float(spb[0]) * float(np.abs(orc.decode_table(fb[0], bool(fb[1]))).max())
            assert np.abs(got[i].astype(np.float64) - ref.astype(np.float64)).max() <= 1e-5 * K * amax * bmax
    if strided:
        full = buf.cpu().numpy()
        assert (full[:, M:, :] == -7.0).all() and (full[:, :, N:] == -7.0).all()      # nothing written outside C
    return cont


@pytest.mark.parametrize("batch,M,N,K", [(1, 5, 7, 9), (3, 197, 197, 64), (4, 197, 64, 197), (2, 128, 256, 128),
                                         (5, 129, 257, 130), (7, 1, 1, 1), (2, 300, 520, 400), (24, 50, 40, 70)])
def test_int8_container_bit_exact(batch, M, N, K):
    assert check(batch, M, N, K, (4, 1), (4, 1), seed=batch + M + N + K) == 0


@pytest.mark.parametrize("fa,fb,cont", [((2, 1), (3, 0), 0), ((5, 0), (4, 1), 1), ((8, 1), (8, 1), 2), ((6, 0), (3, 1), 2)])
def test_other_formats_and_containers(fa, fb, cont):
    assert check(3, 197, 100, 130, fa, fb, seed=fa[0] * 8 + fb[0]) == cont


def test_strided_entries_and_padded_output():
    assert check(3, 70, 36, 100, (4, 1), (4, 0), seed=5, strided=True) == 0
    assert check(2, 200, 132, 64, (8, 1), (8, 1), seed=6, strided=True) == 2


def test_vit_base_attention_shapes_sampled():
    # 12 heads x batch 8: Q K^T and (attention) V, 4-bit; every 7th entry checked in full
    for (M, N, K) in ((197, 197, 64), (197, 64, 197)):
        batch = 96
        a = wl.normal((batch, M, K), seed=M)
        b = wl.normal((batch, N, K), seed=N + 1)
        pa, sa, ca, spa = _quant3(a, (4, 1))
        pb, sb, cb, spb = _quant3(b, (4, 1))
        C, _ = dy.dybit_gemm_batched(M, N, K, pa, (4, 1), sa, pb, (4, 1), sb)
        got = C.cpu().numpy()
        for i in range(0, batch, 7):
            _, ref = orc.gemm(ca[i], (4, 1), spa[0], cb[i], (4, 1), spb[0])
            assert np.array_equal(got[i], ref), i


def test_argument_errors():
    one = torch.tensor([1.0, 1.0], device=DEV)
    A = torch.zeros((2, 8, 16), dtype=torch.uint8, device=DEV)
    B = torch.zeros((3, 8, 16), dtype=torch.uint8, device=DEV)
    with pytest.raises(Exception):
        dy.dybit_gemm_batched(8, 8, 32, A, (4, 1), one, B, (4, 1), one)          # batch mismatch
    with pytest.raises(Exception):
        dy.dybit_gemm_batched(8, 8, 64, A, (4, 1), one, A, (4, 1), one)          # rows too short for K
    assert dy.dybit_gemm_batched_workspace_bytes(0, 8, 8, 8, (4, 1), (4, 1)) == 0
