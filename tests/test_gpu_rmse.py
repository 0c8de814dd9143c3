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
