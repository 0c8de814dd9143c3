"""GPU parity at the sizes and launch configurations bench.py times.

Outputs too large for the oracle to recompute in full are checked on sampled
entries the oracle computes one by one, plus properties that hold at any size
(exact column/row checksums of the integer GEMM, the scale's closed form).
"""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check_packed_samples(x_dev, packed, fmt, scale, rng, n_chunks=48, chunk=8192):
    """Sampled 8192-code windows (aligned so that they start on a byte) + the tail, against the oracle."""
    n = x_dev.numel()
    bits = fmt[0]
    xs = x_dev.reshape(-1)
    # closed form of the scale from the full tensor
    amax = float(xs.abs().max().item())
    m = bits - 1 if fmt[1] else bits
    sp = (np.float32(amax) / np.float32(2.0 ** (m - 1)), np.float32(2.0 ** (m - 1)) / np.float32(amax))
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    starts = [int(s) * 8 for s in rng.integers(0, max(1, (n - chunk) // 8), n_chunks)] + [max(0, (n - chunk) // 8 * 8), 0]
    for s0 in starts:
        cnt = min(chunk, n - s0)
        xh = xs[s0:s0 + cnt].cpu().numpy()
        want = orc.pack(orc.quantize(xh, bits, bool(fmt[1]), sp[1]), bits)
        nbytes = (cnt * bits + 7) // 8
        got = packed[s0 * bits // 8: s0 * bits // 8 + nbytes].cpu().numpy()
        if (cnt * bits) % 8 == 0:
            assert np.array_equal(got, want[:nbytes]), (fmt, s0)
        else:
            assert np.array_equal(got[:-1], want[:nbytes - 1]), (fmt, s0)


@pytest.mark.parametrize("dist,fmt,log2n", [
    ("normal", (4, 1), 28), ("laplace", (2, 1), 26), ("half_normal", (3, 0), 26), ("normal", (6, 1), 26),
    ("laplace", (8, 1), 26), ("half_normal", (8, 0), 24), ("normal", (4, 1), 30),
])
def test_quantize_sweep_sizes_sampled(dist, fmt, log2n):
    n = 1 << log2n
    x = wl.DISTRIBUTIONS[dist]((n,), seed=log2n + fmt[0], device=DEV)
    packed, scale = dy.dybit_quantize_pack(x, fmt)
    assert packed.numel() == dy.dybit_packed_bytes(n, fmt[0])
    _check_packed_samples(x, packed, fmt, scale, np.random.default_rng(log2n))
    # decode(quantize(x)) is within half a code step of x wherever x is inside the range (spot check of the whole tensor)
    back = dy.dybit_decode(packed, n, fmt, scale)
    err = (back - x).abs().max().item()
    top = scale[0].item() * 2.0 ** ((fmt[0] - 1 if fmt[1] else fmt[0]) - 1)
    assert err <= top / 2 + 1e-6
    del x, packed, back
    torch.cuda.empty_cache()


@pytest.mark.parametrize("fmt", [(2, 1), (3, 1), (4, 1), (6, 1), (8, 1)])
@pytest.mark.parametrize("dist", ["normal", "laplace", "half_normal"])
def test_quantize_sweep_2p20_full_parity(fmt, dist):
    n = 1 << 20
    f = fmt if dist != "half_normal" else (fmt[0], 0)
    x = wl.DISTRIBUTIONS[dist]((n,), seed=fmt[0])
    packed, scale = dy.dybit_quantize_pack(x.to(DEV), f)
    sp = orc.absmax_scale(x.numpy(), f[0], bool(f[1]))
    assert np.array_equal(scale.cpu().numpy(), np.array(sp, dtype=np.float32))
    assert np.array_equal(packed.cpu().numpy(), orc.pack(orc.quantize(x.numpy(), f[0], bool(f[1]), sp[1]), f[0]))


def _square_gemm(size, fmt, rng, n_rows, n_cols, n_points):
    a = wl.normal((size, size), seed=size + fmt[0], device=DEV)
    b = wl.normal((size, size), seed=size + fmt[0] + 1, device=DEV)
    pa, sa = dy.dybit_quantize_pack_2d(a, fmt)
    pb, sb = dy.dybit_quantize_pack_2d(b, fmt)
    cont, _, _ = dy.dybit_choose_container(fmt, fmt)
    C, C_raw = dy.dybit_gemm(size, size, size, pa, fmt, sa, pb, fmt, sb, want_raw=(cont == 0))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    # oracle codes of both operands (full), from the same fp32 buffers
    ah, bh = a.cpu().numpy(), b.cpu().numpy()
    del a, b
    spa = orc.absmax_scale(ah, fmt[0], bool(fmt[1]))
    spb = orc.absmax_scale(bh, fmt[0], bool(fmt[1]))
    ca = orc.quantize(ah, fmt[0], bool(fmt[1]), spa[1])
    cb = orc.quantize(bh, fmt[0], bool(fmt[1]), spb[1])
    assert np.array_equal(pa.cpu().numpy(), orc.pack_rows(ca, fmt[0]))
    rows = rng.choice(size, n_rows, replace=False)
    cols = rng.choice(size, n_cols, replace=False)
    ri = np.concatenate([np.repeat(rows, size), np.tile(np.arange(size), n_cols), rng.integers(0, size, n_points)])
    ci = np.concatenate([np.tile(np.arange(size), n_rows), np.repeat(cols, size), rng.integers(0, size, n_points)])
    S, Cref = orc.gemm_sampled(ca, fmt, spa[0], cb, fmt, spb[0], ri, ci)
    got = C[torch.from_numpy(ri).to(DEV), torch.from_numpy(ci).to(DEV)].cpu().numpy()
    if cont == 0:
        got_raw = C_raw[torch.from_numpy(ri).to(DEV), torch.from_numpy(ci).to(DEV)].cpu().numpy()
        assert np.array_equal(got_raw.astype(np.int64), S)
        assert np.array_equal(got, Cref)
        # exact checksums over the whole output: column sums and row sums of the integer GEMM
        m = fmt[0] - 1 if fmt[1] else fmt[0]
        tab = np.round(orc.decode_table(fmt[0], bool(fmt[1])) * 2.0 ** (m - 1)).astype(np.int64)
        IA, IB = tab[ca], tab[cb]
        raw = C_raw.cpu().numpy().astype(np.int64)
        assert np.array_equal(raw.sum(axis=0), IA.sum(axis=0) @ IB.T)
        assert np.array_equal(raw.sum(axis=1), IA @ IB.sum(axis=0))
        del raw, C_raw
        # the call as bench.py times it (no raw sums): same fp32 bits
        C2, _ = dy.dybit_gemm(size, size, size, pa, fmt, sa, pb, fmt, sb)
        torch.cuda.synchronize()
        assert dy.dybit_last_device_status() == (0, 0)
        assert np.array_equal(C2[torch.from_numpy(ri).to(DEV), torch.from_numpy(ci).to(DEV)].cpu().numpy(), Cref)
        assert torch.equal(C, C2)
    else:
        amax = float(spa[0]) * float(np.abs(orc.decode_table(fmt[0], bool(fmt[1]))).max())
        bmax = float(spb[0]) * float(np.abs(orc.decode_table(fmt[0], bool(fmt[1]))).max())
        tol = 1e-5 * size * amax * bmax
        assert np.abs(got.astype(np.float64) - Cref.astype(np.float64)).max() <= tol
        # the whole output through its row and column sums: the exact integer sums of the oracle's definition, scaled,
        # against fp64 sums of the fp32 result; every entry may be off by tol, a sum of `size` entries by size * tol
        m = fmt[0] - 1 if fmt[1] else fmt[0]
        tab = np.round(orc.decode_table(fmt[0], bool(fmt[1])) * 2.0 ** (m - 1)).astype(np.int64)
        IA, IB = tab[ca], tab[cb]
        alpha = float(spa[0]) * float(spb[0]) * 2.0 ** (-2 * (m - 1))
        row_ref = (IA @ IB.sum(axis=0)).astype(np.float64) * alpha
        col_ref = (IA.sum(axis=0) @ IB.T).astype(np.float64) * alpha
        row_got = C.sum(dim=1, dtype=torch.float64).cpu().numpy()
        col_got = C.sum(dim=0, dtype=torch.float64).cpu().numpy()
        assert np.abs(row_got - row_ref).max() <= size * tol
        assert np.abs(col_got - col_ref).max() <= size * tol
        # and far tighter in practice: products are exact in fp32, only the accumulation rounds
        assert np.abs(row_got - row_ref).max() <= 1e-3 * np.abs(row_ref).max() + size * tol * 1e-3
    torch.cuda.empty_cache()


def test_square_gemm_8192_4bit_bench_configuration():
    _square_gemm(8192, (4, 1), np.random.default_rng(1), n_rows=256, n_cols=256, n_points=20000)


@pytest.mark.parametrize("size,fmt", [(1024, (4, 1)), (2048, (4, 1)), (4096, (4, 1)), (1024, (8, 1)), (2048, (8, 1)),
                                      (4096, (8, 1)), (8192, (8, 1))])
def test_square_gemm_sweep(size, fmt):
    # 256 whole rows + 256 whole columns (+ scattered points) against the oracle at every size, both containers
    _square_gemm(size, fmt, np.random.default_rng(size), n_rows=256, n_cols=256, n_points=5000)


def _conv_layer_sampled(L, fx, fw, seed, n_samples=1500, one_call_too=False):
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=seed, device=DEV)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=seed + 1)
    px, sx = dy.dybit_quantize_pack(x, fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    cont, _, _ = dy.dybit_choose_container(fx, fw)
    Y, Y_raw = dy.dybit_conv2d(desc, px, fx, sx, pw, fw, sw, want_raw=(cont == 0))
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    xh = x.cpu().numpy()
    spx = orc.absmax_scale(xh, fx[0], bool(fx[1]))
    spw = orc.absmax_scale(w.numpy(), fw[0], bool(fw[1]))
    assert np.array_equal(sx.cpu().numpy(), np.array(spx, dtype=np.float32))
    cw = orc.quantize(w.numpy(), fw[0], bool(fw[1]), spw[1])
    rng = np.random.default_rng(seed)
    total = Y.numel()
    idx = np.unique(np.concatenate([rng.integers(0, total, n_samples), [0, total - 1],
                                    np.arange(total - L.k, total)]))          # incl. the last output pixel
    S, Yref = orc.conv2d_sampled(xh, fx, spx, cw, fw, spw[0], idx, stride=L.stride, pad=L.pad)
    got = Y.reshape(-1)[torch.from_numpy(idx).to(DEV)].cpu().numpy()
    if cont == 0:
        got_raw = Y_raw.reshape(-1)[torch.from_numpy(idx).to(DEV)].cpu().numpy()
        assert np.array_equal(got_raw.astype(np.int64), S), L.name
        assert np.array_equal(got, Yref), L.name
    else:
        amax = float(spx[0]) * float(np.abs(orc.decode_table(fx[0], bool(fx[1]))).max())
        bmax = float(spw[0]) * float(np.abs(orc.decode_table(fw[0], bool(fw[1]))).max())
        assert np.abs(got.astype(np.float64) - Yref.astype(np.float64)).max() <= 1e-5 * L.gemm_k * amax * bmax, L.name
    if one_call_too:
        # the call bench.py times (fp32 activation in, no raw sums): same codes, same scale, same output bits
        Y1, _, packed1, scale1 = dy.dybit_quantize_conv2d(desc, x, fx, pw, fw, sw)
        torch.cuda.synchronize()
        assert dy.dybit_last_device_status() == (0, 0)
        assert torch.equal(packed1, px) and torch.equal(scale1, sx), L.name
        assert torch.equal(Y1, Y), L.name
    return cont


def _distinct(layers):
    seen, out = set(), []
    for i, L in enumerate(layers):
        key = (L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad)
        if key not in seen:
            seen.add(key)
            out.append((i, L))
    return out


@pytest.mark.parametrize("i,L", _distinct(wl.resnet18_layers(32)), ids=lambda v: getattr(v, "name", str(v)))
def test_resnet18_batch32_uniform_4bit_sampled(i, L):
    assert _conv_layer_sampled(L, (4, 0), (4, 1), seed=1000 + i, one_call_too=True) == 0


def test_resnet18_batch32_folded_step_in_the_bench_launch_configuration():
    """The step as bench.py times it: dybit_quantize_expand_layers over all 21 layers, then the tensor-core work, first as
    dybit_conv2d_prepared per layer round-robin on three streams, then as dybit_conv2d_prepared_layers (shared
    launches; the form the bench uses).  Every layer's codes, scale and output must equal, bit for bit, what the
    one-layer call gives (which the test above checks against the oracle), and sampled outputs of four layers are
    checked against the oracle directly."""
    layers = wl.resnet18_layers(32)
    fx, fw = (4, 0), (4, 1)
    args, ws = [], []
    for i, L in enumerate(layers):
        x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i, device=DEV)
        w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2000 + i)
        pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
        args.append(dict(desc=dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1), X=x, fx=fx, W=pw, fw=fw,
                         scale_w=sw))
        ws.append(w)
    folded = dy.ConvLayers(args)
    side = [torch.cuda.Stream(DEV) for _ in range(3)]
    cur = torch.cuda.current_stream()
    n0 = dy.dybit_launch_count()
    dy.dybit_quantize_expand_layers(folded)
    for st in side:
        st.wait_stream(cur)
    for j in range(len(layers)):
        dy.dybit_conv2d_prepared(folded, j, stream=side[j % 3])
    for st in side:
        cur.wait_stream(st)
    torch.cuda.synchronize()
    assert dy.dybit_launch_count() - n0 == 2 + len(layers)
    assert dy.dybit_last_device_status() == (0, 0)
    per_layer = [y.clone() for y in folded.Y]
    for y in folded.Y:
        y.zero_()
    n1 = dy.dybit_launch_count()
    dy.dybit_conv2d_prepared_layers(folded)
    torch.cuda.synchronize()
    assert dy.dybit_launch_count() - n1 <= 8
    assert dy.dybit_last_device_status() == (0, 0)
    for i, L in enumerate(layers):
        assert torch.equal(per_layer[i], folded.Y[i]), L.name
    del per_layer
    for i, (L, a) in enumerate(zip(layers, args)):
        Y1, _, p1, s1 = dy.dybit_quantize_conv2d(a["desc"], a["X"], fx, a["W"], fw, a["scale_w"])
        assert torch.equal(p1, folded.packed[i]) and torch.equal(s1, folded.scale[i]), L.name
        assert torch.equal(Y1, folded.Y[i]), L.name
        del Y1, p1
    for i in (0, 1, 11, 20):
        L = layers[i]
        xh = args[i]["X"].cpu().numpy()
        spx = orc.absmax_scale(xh, 4, False)
        spw = orc.absmax_scale(ws[i].numpy(), 4, True)
        cw = orc.quantize(ws[i].numpy(), 4, True, spw[1])
        total = folded.Y[i].numel()
        idx = np.unique(np.concatenate([np.random.default_rng(i).integers(0, total, 400), [0, total - 1]]))
        _, y_ref = orc.conv2d_sampled(xh, fx, spx, cw, fw, spw[0], idx, stride=L.stride, pad=L.pad)
        got = folded.Y[i].reshape(-1)[torch.from_numpy(idx).to(DEV)].cpu().numpy()
        assert np.array_equal(got, y_ref), L.name
    del folded
    torch.cuda.empty_cache()


_R50 = wl.resnet50_layers(64)
_R50_BITS = wl.mixed_bitwidths(len(_R50), seed=0)


@pytest.mark.parametrize("i,L", _distinct(_R50), ids=lambda v: getattr(v, "name", str(v)))
def test_resnet50_batch64_mixed_bitwidths_sampled(i, L):
    wbits, abits = _R50_BITS[i]
    _conv_layer_sampled(L, (abits, 0), (wbits, 1), seed=3000 + i, n_samples=800)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("i,L", _distinct(wl.resnet18_layers(32)), ids=lambda v: getattr(v, "name", str(v)))
def test_resnet18_batch32_requant_epilogue_sampled(i, L):
    """Bench-size layers through the re-quantizing epilogue: sampled output codes against the oracle
    (sampled conv -> ReLU -> encode with the given output scale)."""
    fx, fw, fq = (4, 0), (4, 1), (4, 0)
    x = wl.half_normal((L.n, L.h, L.w, L.c), seed=1000 + i, device=DEV)
    w = wl.kaiming_normal(L.k, L.r, L.s, L.c, seed=2000 + i)
    px, sx = dy.dybit_quantize_pack(x, fx)
    pw, sw = dy.dybit_quantize_pack_2d(w.reshape(L.k, -1).to(DEV), fw)
    xh = x.cpu().numpy()
    spx = orc.absmax_scale(xh, 4, False)
    spw = orc.absmax_scale(w.numpy(), 4, True)
    cw = orc.quantize(w.numpy(), 4, True, spw[1])
    total = L.gemm_m * L.k
    rng = np.random.default_rng(i)
    idx = np.unique(np.concatenate([rng.integers(0, total, 1200), [0, total - 1]]))
    _, yref = orc.conv2d_sampled(xh, fx, spx, cw, fw, spw[0], idx, stride=L.stride, pad=L.pad)
    # output scale from the sampled activations (a stand-in for a calibrated scale); some samples saturate
    sq = orc.absmax_scale(np.maximum(yref, 0) * 0.8, 4, False)
    scale_q = torch.tensor([float(sq[0]), float(sq[1])], dtype=torch.float32, device=DEV)
    desc = dy.ConvDesc(L.n, L.h, L.w, L.c, L.k, L.r, L.s, L.stride, L.pad, 1)
    Q = dy.dybit_conv2d_requant(desc, px, fx, sx, pw, fw, sw, fq, scale_q, relu=True)
    torch.cuda.synchronize()
    assert dy.dybit_last_device_status() == (0, 0)
    qb = Q.cpu().numpy()
    got = (qb[idx // 2] >> ((idx % 2) * 4)) & 0xF                    # 4-bit codes: two per byte, low nibble first
    want = orc.quantize(np.maximum(yref, 0), 4, False, sq[1])
    assert np.array_equal(got, want), L.name
