"""GPU parity of the Eq. 2 error metric against the oracle (fp64 sums in a different order: 1e-9 relative)."""
import numpy as np
import pytest
import torch

import paper_2302_12510_b200 as dy
from paper_2302_12510_b200 import workloads as wl
from oracle import dybit_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("fmt", [(b, s) for b in range(2, 9) for s in (0, 1)])
@pytest.mark.parametrize("n,dist", [(1, "normal"), (1000, "laplace"), (262144 + 77, "normal"), (50001, "half_normal")])
def test_rmse_matches_oracle(fmt, n, dist):
    x = wl.DISTRIBUTIONS[dist]((n,), seed=n + fmt[0]) + 0.25
    scale = dy.dybit_absmax_scale(x.to(DEV), fmt)
    out = dy.dybit_rmse(x.to(DEV), fmt, scale).cpu().numpy()
    sp = orc.absmax_scale(x.numpy(), fmt[0], bool(fmt[1]))
    r, sigma, mse = orc.rmse(x.numpy(), fmt[0], bool(fmt[1]), sp)
    assert out[3] == n
    assert out[1] == pytest.approx(sigma, rel=1e-9, abs=1e-300)
    assert out[2] == pytest.approx(mse, rel=1e-9, abs=1e-300)
    assert out[0] == pytest.approx(r, rel=1e-9, abs=1e-300)


def test_rmse_degenerate_and_unaligned():
    fmt = (4, 1)
    one = torch.tensor([1.0, 1.0], device=DEV)
    assert dy.dybit_rmse(torch.zeros(0, device=DEV), fmt, one).tolist() == [0.0, 0.0, 0.0, 0.0]
    out = dy.dybit_rmse(torch.full((1000,), 0.3, device=DEV), fmt, one).cpu().numpy()
    assert out[0] == 0.0 and out[1] == 0.0                    # constant tensor: sigma is exactly 0
    base = wl.normal((10001,), 3)
    xd = base.to(DEV)[1:]
    sp = orc.absmax_scale(base[1:].numpy(), 4, True)
    scale = torch.tensor([float(sp[0]), float(sp[1])], device=DEV)
    out = dy.dybit_rmse(xd, fmt, scale).cpu().numpy()
    assert out[0] == pytest.approx(orc.rmse(base[1:].numpy(), 4, True, sp)[0], rel=1e-9)


def test_rmse_large_tensor_and_bitwidth_ordering():
    n = 1 << 24
    x = wl.normal((n,), 5, device=DEV)
    errs = []
    for bits in (2, 4, 8):
        scale = dy.dybit_absmax_scale(x, (bits, 1))
        errs.append(dy.dybit_rmse(x, (bits, 1), scale)[0].item())
    assert errs[0] > errs[1] > errs[2] > 0
    xh = x[: 1 << 20].cpu().numpy()
    sp = orc.absmax_scale(xh, 4, True)
    scale = torch.tensor([float(sp[0]), float(sp[1])], device=DEV)
    got = dy.dybit_rmse(x[: 1 << 20], (4, 1), scale).cpu().numpy()
    assert got[0] == pytest.approx(orc.rmse(xh, 4, True, sp)[0], rel=1e-9)


def _scales_tensor(pairs):
    return torch.tensor([[float(a), float(b)] for a, b in pairs], dtype=torch.float32, device=DEV)


@pytest.mark.parametrize("n,dist", [(1, "normal"), (7, "laplace"), (262144 + 77, "normal"), (50001, "half_normal")])
def test_rmse_sweep_all_formats_in_two_passes_matches_oracle(n, dist):
    # every format the library has, 14 candidates, split over two calls of 7 and one call of 14
    x = wl.DISTRIBUTIONS[dist]((n,), seed=n) + 0.25
    fmts = [(b, s) for b in range(2, 9) for s in (0, 1)]
    pairs = [orc.absmax_scale(x.numpy(), b, bool(s)) for b, s in fmts]
    want = [orc.rmse(x.numpy(), b, bool(s), sp) for (b, s), sp in zip(fmts, pairs)]
    xd = x.to(DEV)
    for lo, hi in ((0, 7), (7, 14), (0, 14)):
        out, best = dy.dybit_rmse_sweep(xd, fmts[lo:hi], _scales_tensor(pairs[lo:hi]))
        out = out.cpu().numpy()
        for row, (r, sigma, mse) in zip(out, want[lo:hi]):
            assert row[3] == n
            assert row[1] == pytest.approx(sigma, rel=1e-9, abs=1e-300)
            assert row[2] == pytest.approx(mse, rel=1e-9, abs=1e-300)
            assert row[0] == pytest.approx(r, rel=1e-9, abs=1e-300)
        assert int(best.item()) == int(np.argmin(out[:, 0]))


def test_rmse_sweep_scale_search_finds_the_clipping_ratio_the_oracle_finds():
    # 16 candidate scales for one format: the max-abs scale shrunk by clipping ratios 1.0 ... 0.25
    n, fmt = 300001, (4, 1)
    x = wl.laplace((n,), seed=21)
    base = orc.absmax_scale(x.numpy(), fmt[0], True)
    ratios = np.linspace(1.0, 0.25, 16).astype(np.float32)
    pairs = [(np.float32(base[0]) * r, np.float32(1.0) / (np.float32(base[0]) * r)) for r in ratios]
    want = np.array([orc.rmse(x.numpy(), fmt[0], True, p)[0] for p in pairs])
    out, best = dy.dybit_rmse_sweep(x.to(DEV), [fmt] * 16, _scales_tensor(pairs))
    got = out.cpu().numpy()[:, 0]
    assert np.allclose(got, want, rtol=1e-9, atol=0)
    assert int(best.item()) == int(np.argmin(want))
    assert 0 < int(best.item()) < 15                  # clipping the Laplace tail does pay, but not without limit
    # one candidate of the sweep is the single-candidate entry point
    one = dy.dybit_rmse(x.to(DEV), fmt, _scales_tensor(pairs[3:4]).reshape(2)).cpu().numpy()
    assert one[0] == pytest.approx(got[3], rel=1e-12)


def test_rmse_sweep_degenerate_unaligned_and_errors():
    fmts = [(4, 1), (2, 0), (8, 1)]
    ones = _scales_tensor([(1.0, 1.0)] * 3)
    out, best = dy.dybit_rmse_sweep(torch.zeros(0, device=DEV), fmts, ones)
    assert out.cpu().numpy().tolist() == [[0.0] * 4] * 3 and int(best.item()) == 0
    out, best = dy.dybit_rmse_sweep(torch.full((1000,), 0.3, device=DEV), fmts, ones)
    assert (out.cpu().numpy()[:, :2] == 0).all() and int(best.item()) == 0      # constant tensor: sigma exactly 0
    base = wl.normal((10003,), 3)
    for off in (1, 2, 3):
        xs = base[off:]
        pairs = [orc.absmax_scale(xs.numpy(), b, bool(s)) for b, s in fmts]
        out, _ = dy.dybit_rmse_sweep(base.to(DEV)[off:], fmts, _scales_tensor(pairs))
        for row, (b, s), sp in zip(out.cpu().numpy(), fmts, pairs):
            assert row[0] == pytest.approx(orc.rmse(xs.numpy(), b, bool(s), sp)[0], rel=1e-9)
    with pytest.raises(Exception):
        dy.dybit_rmse_sweep(base.to(DEV), [(4, 1)] * 17, _scales_tensor([(1.0, 1.0)] * 17))
    with pytest.raises(Exception):
        dy.dybit_rmse_sweep(base.to(DEV), [(9, 1)], _scales_tensor([(1.0, 1.0)]))
    with pytest.raises(Exception):
        dy.dybit_rmse_sweep(base.to(DEV), [], torch.zeros(0, device=DEV))
