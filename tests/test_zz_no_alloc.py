"""dybit_gemm_static_ws: the GEMM entry point for callers that cannot allocate device memory
(fixed start-up memory budget, plug-in inside an application that owns the GPU's memory, a path
where an allocator call is not allowed).  Its scratch is an array inside the library; this test
checks, through the C ABI, that it returns exactly what dybit_gemm returns -- twice in a row with
different operands, since every call reuses the same scratch bytes -- and that it refuses problems
larger than the built-in scratch.

Collected last (file name) so that a run stopping at the first failure has finished all other tests."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _operands(M, N, K, fa, fb, seed):
    a = wl.normal((M, K), seed=seed)
    b = wl.normal((N, K), seed=seed + 1)
    if not fa[1]:
        a = a.abs()
    if not fb[1]:
        b = b.abs()
    pa, sa = dy.dybit_quantize_pack_2d(a.to(DEV), fa)
    pb, sb = dy.dybit_quantize_pack_2d(b.to(DEV), fb)
    return pa, sa, pb, sb


@pytest.mark.parametrize("fa,fb", [((4, 1), (4, 0)), ((8, 1), (8, 1))])
def test_static_scratch_gemm_matches_workspace_gemm_twice(fa, fb):
    cont, _, _ = dy.dybit_choose_container(fa, fb)
    # second problem is smaller and differently shaped: stale bytes of the first stay in the scratch
    for call, (M, N, K) in enumerate([(300, 520, 400), (129, 257, 131)]):
        pa, sa, pb, sb = _operands(M, N, K, fa, fb, seed=10 * call + fa[0])
        want, want_raw = dy.dybit_gemm(M, N, K, pa, fa, sa, pb, fb, sb, want_raw=(cont == 0))
        got = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
        got_raw = torch.full((M, N), -1, dtype=torch.int32, device=DEV) if cont == 0 else None
        dy.dybit_gemm_static_ws(M, N, K, pa, fa, sa, pb, fb, sb, got, got_raw)
        torch.cuda.synchronize()
        assert dy.dybit_last_device_status() == (0, 0)
        # same kernels on the same expanded operands: identical bits, which is inside every tolerance
        # the GEMM tests use (exact for int8, 1e-5*K*max|a|*max|b| for the floating containers)
        assert torch.equal(got, want)
        if cont == 0:
            assert torch.equal(got_raw, want_raw)


def test_static_scratch_gemm_matches_the_oracle_and_allocates_nothing():
    # against the CPU oracle directly (not only against dybit_gemm), and with the allocator's books and the
    # device's free memory read before and after a call: the entry point must leave both untouched
    fa, fb = (4, 0), (4, 1)
    M, N, K = 200, 136, 333
    a = wl.half_normal((M, K), seed=31)
    b = wl.normal((N, K), seed=32, std=0.05)
    pa, sa = dy.dybit_quantize_pack_2d(a.to(DEV), fa)
    pb, sb = dy.dybit_quantize_pack_2d(b.to(DEV), fb)
    got = torch.empty((M, N), dtype=torch.float32, device=DEV)
    got_raw = torch.empty((M, N), dtype=torch.int32, device=DEV)
    dy.dybit_gemm_static_ws(M, N, K, pa, fa, sa, pb, fb, sb, got, got_raw)       # first call on this device: set-up
    torch.cuda.synchronize()
    allocated, reserved, free = torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]
    dy.dybit_gemm_static_ws(M, N, K, pa, fa, sa, pb, fb, sb, got, got_raw)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == allocated and torch.cuda.memory_reserved() == reserved
    assert torch.cuda.mem_get_info()[0] == free
    spa, spb = orc.absmax_scale(a.numpy(), 4, False), orc.absmax_scale(b.numpy(), 4, True)
    S, C_ref = orc.gemm(orc.quantize(a.numpy(), 4, False, spa[1]), fa, spa[0],
                        orc.quantize(b.numpy(), 4, True, spb[1]), fb, spb[0])
    assert np.array_equal(got_raw.cpu().numpy().astype(np.int64), S)
    assert np.array_equal(got.cpu().numpy(), C_ref)


def test_static_scratch_gemm_refuses_oversized_problems():
    fa = fb = (4, 1)
    M = N = K = 4096                     # needs 2 * 16 MiB of expanded operands
    assert dy.dybit_gemm_workspace_bytes(M, N, K, fa, fb) > dy.STATIC_WS_BYTES
    rs = dy.dybit_row_stride_bytes(K, 4)
    pa = torch.zeros((M, rs), dtype=torch.uint8, device=DEV)
    one = torch.tensor([1.0, 1.0], device=DEV)
    out = torch.zeros((M, N), dtype=torch.float32, device=DEV)
    launches = dy.dybit_launch_count()
    with pytest.raises(dy.DybitError) as e:
        dy.dybit_gemm_static_ws(M, N, K, pa, fa, one, pa, fb, one, out)
    assert e.value.status == 4
    assert dy.dybit_launch_count() == launches          # nothing was launched
