"""The give-up path of the bounded device-side waits, exercised in the one safe form: a wait, with the library's own
routine and a 1 ms limit, on a barrier that nothing ever signals.  The kernel must return by itself, the status word must
report the timeout exactly once, and the device must keep producing bit-exact results afterwards."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DYBIT_ERR_DEVICE_TIMEOUT = 6


def _gemm_against_oracle():
    fx, fw = (4, 0), (4, 1)
    x = wl.half_normal((96, 300), seed=4)
    w = wl.normal((72, 300), seed=5, std=0.02)
    px, sx = dy.dybit_quantize_pack_2d(x.to(DEV), fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.to(DEV), fw)
    C, C_raw = dy.dybit_gemm(96, 72, 300, px, fx, sx, pw, fw, sw, want_raw=True)
    spx, spw = orc.absmax_scale(x.numpy(), 4, False), orc.absmax_scale(w.numpy(), 4, True)
    S, C_ref = orc.gemm(orc.quantize(x.numpy(), 4, False, spx[1]), fx, spx[0],
                        orc.quantize(w.numpy(), 4, True, spw[1]), fw, spw[0])
    assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S)
    assert np.array_equal(C.cpu().numpy(), C_ref)


def test_bounded_wait_runs_out_and_is_reported_once():
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    result = dy.dybit_selftest_wait_timeout(1_000_000)          # 1 ms
    t1.record()
    torch.cuda.synchronize()
    assert result.tolist() == [1, 1]                            # the wait failed and raised the CTA's abort flag
    ms = t0.elapsed_time(t1)
    assert 0.9 <= ms < 50.0, ms                                 # it waited for its limit, not for ever
    status, detail = dy.dybit_last_device_status()
    assert status == DYBIT_ERR_DEVICE_TIMEOUT
    assert detail == (0x5E << 8) | 1                            # site code of the self-test, "a wait expired" bit
    assert dy.dybit_last_device_status() == (0, 0)              # reading the word cleared it
    _gemm_against_oracle()                                      # the context is intact
    assert dy.dybit_last_device_status() == (0, 0)


def test_selftest_argument_errors():
    with pytest.raises(dy.DybitError):
        dy.dybit_selftest_wait_timeout(0)
    with pytest.raises(dy.DybitError):
        dy.dybit_selftest_wait_timeout(10**9)                   # limits above 0.1 s are refused
