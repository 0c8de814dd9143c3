"""GPU parity of the fake-quantization pair against the oracle: bit-exact fp32 in both directions."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _same_bits(a: np.ndarray, b: np.ndarray) -> bool:
    return np.array_equal(a.view(np.uint32), b.view(np.uint32))


@pytest.mark.parametrize("fmt", [(b, s) for b in range(2, 9) for s in (0, 1)])
@pytest.mark.parametrize("n,dist", [(1, "normal"), (1003, "laplace"), (262144 + 77, "normal")])
def test_forward_matches_decode_of_encode(fmt, n, dist):
    x = wl.DISTRIBUTIONS[dist]((n,), seed=n + fmt[0] + 20)
    sp = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    scale = torch.tensor([float(sp[0]), float(sp[1])], dtype=torch.float32, device=DEV)
    y = dy.dybit_fake_quant(x.to(DEV), fmt, scale).cpu().numpy()
    assert _same_bits(y, orc.fake_quant(x.numpy(), fmt[0], bool(fmt[1]), sp))


@pytest.mark.parametrize("fmt", [(4, 1), (4, 0), (8, 1), (2, 1), (5, 0)])
def test_forward_midpoints_specials_and_clipping_scale(fmt):
    # every midpoint between neighbouring values and its fp32 neighbours, specials, and a scale that clips
    tab = np.unique(np.abs(orc.decode_table(fmt[0], bool(fmt[1])).astype(np.float64)))
    mids = ((tab[1:] + tab[:-1]) / 2).astype(np.float32)
    pts = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf)),
                          tab.astype(np.float32)])
    x = np.concatenate([pts, -pts, np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 3e38, -3e38],
                                            dtype=np.float32)]).astype(np.float32)
    for sp in ((1.0, 1.0), (0.37, float(np.float32(1.0) / np.float32(0.37)))):
        scale = torch.tensor([sp[0], sp[1]], dtype=torch.float32, device=DEV)
        xs = (x * np.float32(sp[0])).astype(np.float32)
        y = dy.dybit_fake_quant(torch.from_numpy(xs).to(DEV), fmt, scale).cpu().numpy()
        assert _same_bits(y, orc.fake_quant(xs, fmt[0], bool(fmt[1]), sp))


def test_forward_in_place_unaligned_and_empty():
    fmt = (4, 1)
    base = wl.normal((20011,), 9)
    sp = orc.absmax_scale(base.numpy(), 4, True)
    scale = torch.tensor([float(sp[0]), float(sp[1])], dtype=torch.float32, device=DEV)
    for off in (1, 2, 3):
        xd = base.to(DEV)[off:]
        y = dy.dybit_fake_quant(xd, fmt, scale)
        want = orc.fake_quant(base[off:].numpy(), 4, True, sp)
        assert _same_bits(y.cpu().numpy(), want)
        # different 16-byte phases of source and destination
        buf = torch.empty(base.numel() + 4, dtype=torch.float32, device=DEV)
        out = buf[(off + 1) % 4:][: xd.numel()]
        dy.dybit_fake_quant(xd, fmt, scale, out=out)
        assert _same_bits(out.cpu().numpy(), want)
        dy.dybit_fake_quant(xd, fmt, scale, out=xd)               # in place
        assert _same_bits(xd.cpu().numpy(), want)
    assert dy.dybit_fake_quant(torch.zeros(0, device=DEV), fmt, scale).numel() == 0


@pytest.mark.parametrize("fmt", [(4, 1), (4, 0), (2, 1), (8, 0)])
@pytest.mark.parametrize("n", [1, 1001, 262144 + 5])
def test_backward_matches_oracle(fmt, n):
    x = wl.normal((n,), seed=n + fmt[0])
    g = wl.normal((n,), seed=n + fmt[0] + 1)
    full = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    for shrink in (1.0, 0.3):
        s0 = np.float32(full[0]) * np.float32(shrink)
        sp = (float(s0), float(np.float32(1.0) / s0))
        scale = torch.tensor([sp[0], sp[1]], dtype=torch.float32, device=DEV)
        gx = dy.dybit_fake_quant_backward(x.to(DEV), g.to(DEV), fmt, scale).cpu().numpy()
        assert _same_bits(gx, orc.fake_quant_backward(x.numpy(), g.numpy(), fmt[0], bool(fmt[1]), sp))


def test_backward_range_ends_nan_and_unaligned():
    fmt, sp = (4, 1), (0.5, 2.0)                                   # covers [-2, 2]
    scale = torch.tensor(sp, dtype=torch.float32, device=DEV)
    x = np.array([-2.0000002, -2.0, 2.0, 2.0000002, np.nan, 0.0, np.inf, -np.inf, 1.0], dtype=np.float32)
    g = np.arange(1, 10, dtype=np.float32)
    gx = dy.dybit_fake_quant_backward(torch.from_numpy(x).to(DEV), torch.from_numpy(g).to(DEV), fmt, scale)
    assert gx.cpu().numpy().tolist() == [0, 2, 3, 0, 0, 6, 0, 0, 9]
    base, gb = wl.normal((10007,), 1), wl.normal((10007,), 2)
    for off in (1, 3):
        gx = dy.dybit_fake_quant_backward(base.to(DEV)[off:], gb.to(DEV)[off:], fmt, scale).cpu().numpy()
        assert _same_bits(gx, orc.fake_quant_backward(base[off:].numpy(), gb[off:].numpy(), 4, True, sp))
