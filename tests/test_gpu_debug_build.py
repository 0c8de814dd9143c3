"""The range-checked debug build (libdybit_debug.so, -DDYBIT_DEBUG_BOUNDS): the same sources with every global store
whose extent the kernel knows wrapped in a check that skips the access and records a status code instead of
trapping.  Run in a child process (the library is chosen at import time): a pass over the hot path must give the
oracle's bits and leave the status word clean, i.e. no check fires on in-range work."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import numpy as np, torch
import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl, binding, _build
from oracle import dybit_oracle as orc
assert binding.lib._name == _build.DEBUG_LIB_PATH, binding.lib._name
dev = "cuda:0"
for fx, fw in (((4, 0), (4, 1)), ((3, 1), (5, 1)), ((8, 0), (8, 1))):
    for (M, N, K) in ((64, 256, 256), (129, 77, 1000)):
        a = wl.normal((M, K), seed=M); b = wl.normal((N, K), seed=N)
        if not fx[1]: a = a.abs()
        pa, sa = dy.dybit_quantize_pack_2d(a.to(dev), fx); pb, sb = dy.dybit_quantize_pack_2d(b.to(dev), fw)
        cont, _, _ = dy.dybit_choose_container(fx, fw)
        C, C_raw = dy.dybit_gemm(M, N, K, pa, fx, sa, pb, fw, sb, want_raw=(cont == 0))
        spa, spb = orc.absmax_scale(a.numpy(), fx[0], bool(fx[1])), orc.absmax_scale(b.numpy(), fw[0], bool(fw[1]))
        ca, cb = orc.quantize(a.numpy(), fx[0], bool(fx[1]), spa[1]), orc.quantize(b.numpy(), fw[0], bool(fw[1]), spb[1])
        assert np.array_equal(pa.cpu().numpy(), orc.pack_rows(ca, fx[0]))
        S, C_ref = orc.gemm(ca, fx, spa[0], cb, fw, spb[0])
        if cont == 0:
            assert np.array_equal(C_raw.cpu().numpy().astype(np.int64), S) and np.array_equal(C.cpu().numpy(), C_ref)
x = wl.normal((50000 + 3,), seed=9)
for fmt in ((2, 1), (4, 1), (5, 0), (8, 1)):
    xx = x.abs() if not fmt[1] else x
    packed, scale = dy.dybit_quantize_pack(xx.to(dev), fmt)
    sp = orc.absmax_scale(xx.numpy(), fmt[0], bool(fmt[1]))
    assert np.array_equal(packed.cpu().numpy(), orc.pack(orc.quantize(xx.numpy(), fmt[0], bool(fmt[1]), sp[1]), fmt[0]))
    back = dy.dybit_decode(packed, xx.numel(), fmt, scale)
    assert np.array_equal(back.cpu().numpy(), orc.dequantize(orc.quantize(xx.numpy(), fmt[0], bool(fmt[1]), sp[1]), fmt[0], bool(fmt[1]), sp[0]))
for L in (wl.ConvLayer("a", 2, 14, 14, 64, 64, 3, 3, 1, 1), wl.ConvLayer("b", 2, 32, 32, 3, 64, 7, 7, 2, 3), wl.ConvLayer("c", 3, 9, 9, 128, 40, 3, 3, 2, 1)):
    xa = wl.half_normal((L.n, L.h, L.w, L.c), seed=1); wa = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2)
    pw, sw = dy.dybit_quantize_pack_2d(wa.reshape(L.k, -1).to(dev), (4, 1))
    d = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Y, Y_raw, packed, scale = dy.dybit_quantize_conv2d(d, xa.to(dev), (4, 0), pw, (4, 1), sw, want_raw=True)
    sa_, sb_ = orc.absmax_scale(xa.numpy(), 4, False), orc.absmax_scale(wa.numpy(), 4, True)
    Sc, Yc = orc.conv2d(orc.quantize(xa.numpy(), 4, False, sa_[1]), (4, 0), sa_[0], orc.quantize(wa.numpy(), 4, True, sb_[1]), (4, 1), sb_[0], stride=L.stride, pad=L.pad)
    assert np.array_equal(Y_raw.cpu().numpy().astype(np.int64), Sc) and np.array_equal(Y.cpu().numpy(), Yc)
# the same three layers through the folded launches (absmax_layers_kernel, quantize_expand_layers_kernel)
args, want = [], []
for L in (wl.ConvLayer("a", 2, 14, 14, 64, 64, 3, 3, 1, 1), wl.ConvLayer("b", 2, 32, 32, 3, 64, 7, 7, 2, 3), wl.ConvLayer("c", 3, 9, 9, 128, 40, 3, 3, 2, 1)):
    xa = wl.half_normal((L.n, L.h, L.w, L.c), seed=1); wa = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2)
    pw, sw = dy.dybit_quantize_pack_2d(wa.reshape(L.k, -1).to(dev), (4, 1))
    d = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    args.append(dict(desc=d, X=xa.to(dev), fx=(4, 0), W=pw, fw=(4, 1), scale_w=sw, want_raw=True))
    sa_, sb_ = orc.absmax_scale(xa.numpy(), 4, False), orc.absmax_scale(wa.numpy(), 4, True)
    want.append(orc.conv2d(orc.quantize(xa.numpy(), 4, False, sa_[1]), (4, 0), sa_[0], orc.quantize(wa.numpy(), 4, True, sb_[1]), (4, 1), sb_[0], stride=L.stride, pad=L.pad))
layers = dy.ConvLayers(args)
dy.dybit_quantize_expand_layers(layers)
for i in range(len(args)):
    Y, Y_raw = dy.dybit_conv2d_prepared(layers, i)
    assert np.array_equal(Y_raw.cpu().numpy().astype(np.int64), want[i][0]) and np.array_equal(Y.cpu().numpy(), want[i][1])
dy.dybit_conv2d_prepared_layers(layers)
for i in range(len(args)):
    assert np.array_equal(layers.raw[i].cpu().numpy().astype(np.int64), want[i][0]) and np.array_equal(layers.Y[i].cpu().numpy(), want[i][1])
torch.cuda.synchronize()
assert dy.dybit_last_device_status() == (0, 0), dy.dybit_last_device_status()
print("debug build ok")
"""


def test_debug_build_gives_the_oracles_bits_and_no_check_fires():
    from paper_2302_12510_b200 import _build
    if not os.path.exists(_build.DEBUG_LIB_PATH):
        _build.build_library(debug_bounds=True)
    env = dict(os.environ, DYBIT_LIBRARY="debug", PYTHONPATH=ROOT)
    proc = subprocess.run([sys.executable, "-c", SCRIPT], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert proc.returncode == 0, proc.stdout[-2000:] + proc.stderr[-4000:]
    assert "debug build ok" in proc.stdout
