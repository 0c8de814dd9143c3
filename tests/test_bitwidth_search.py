"""Algorithm 1: the oracle's plain Python search against facts that hold for any correct run, a hand-traced case,
and the library's host implementation (dybit_search_bitwidths) on random tables."""
import itertools

import numpy as np
import pytest

import paper_2302_12510_b200 as dy
from oracle import bitwidth_search as bs

LEVELS = (8, 4, 2)


def _tables(n, seed):
    rng = np.random.default_rng(seed)
    lat, rmse = [], []
    for _ in range(n):
        base_l, base_r = rng.uniform(1, 10), rng.uniform(0.01, 0.1)
        L, R = {}, {}
        for a, w in itertools.product(LEVELS, LEVELS):
            # fewer bits: faster (ideally x (8/a)(8/w), Section III-B.3) and less accurate
            L[(a, w)] = base_l / ((8 / a) * (8 / w)) ** rng.uniform(0.6, 1.0)
            R[(a, w)] = base_r * (1 + (8 / a - 1) * rng.uniform(0.5, 2) + (8 / w - 1) * rng.uniform(0.5, 2))
        lat.append(L)
        rmse.append(R)
    return lat, rmse


def _tot(t, W, A):
    return sum(t[i][(A[i], W[i])] for i in range(len(W)))


def test_hand_traced_speedup_case():
    # two layers; layer 0 is slow and error-tolerant, layer 1 fast and fragile; k = 1, alpha = 2
    lat = [{(a, w): 8.0 / ((8 / a) * (8 / w)) for a in LEVELS for w in LEVELS},
           {(a, w): 2.0 / ((8 / a) * (8 / w)) for a in LEVELS for w in LEVELS}]
    rmse = [{(a, w): 0.01 * (8 / a) * (8 / w) for a in LEVELS for w in LEVELS},
            {(a, w): 0.10 * (8 / a) * (8 / w) for a in LEVELS for w in LEVELS}]
    # start (8,8),(8,8): total 10.  Iteration 1: slowest = layer 0; W0 8->4: total 4+2 = 6, 2*6 > 10, not met;
    # A0 8->4: total 2+2 = 4, 2*4 <= 10 -> met.
    W, A = bs.search(lat, rmse, "speedup", 2.0, 1)
    assert (W, A) == ([4, 8], [4, 8])


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("alpha", [1.5, 3.0, 6.0])
def test_speedup_search_meets_eq3_or_bottoms_out(seed, alpha):
    lat, rmse = _tables(7, seed)
    W, A = bs.search(lat, rmse, "speedup", alpha, 3)
    assert all(b in LEVELS for b in W + A)
    base = _tot(lat, [8] * 7, [8] * 7)
    assert alpha * _tot(lat, W, A) <= base or (set(W) == {2} and set(A) == {2})
    # a larger alpha never leaves more bits
    W2, A2 = bs.search(lat, rmse, "speedup", alpha * 1.5, 3)
    assert sum(W2) + sum(A2) <= sum(W) + sum(A)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("beta", [1.2, 2.0, 5.0])
def test_rmse_search_stays_inside_the_eq4_budget(seed, beta):
    lat, rmse = _tables(6, seed + 10)
    W, A = bs.search(lat, rmse, "rmse", beta, 2)
    base = _tot(rmse, [8] * 6, [8] * 6)
    assert _tot(rmse, W, A) <= beta * base
    assert _tot(lat, W, A) <= _tot(lat, [8] * 6, [8] * 6)


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("strategy,c,k", [("speedup", 2.5, 1), ("speedup", 5.0, 4), ("rmse", 1.8, 2), ("rmse", 4.0, 3)])
def test_library_search_equals_oracle(seed, strategy, c, k):
    n = 9
    lat, rmse = _tables(n, seed + 100)
    W, A = bs.search(lat, rmse, strategy, c, k)
    flat = lambda t: [t[i][(a, w)] for i in range(n) for a in LEVELS for w in LEVELS]   # noqa: E731
    Wl, Al = dy.dybit_search_bitwidths(flat(lat), flat(rmse), n, strategy, c, k)
    assert (Wl, Al) == (W, A)


def test_library_search_argument_errors():
    with pytest.raises(dy.DybitError):
        dy.dybit_search_bitwidths([1.0] * 9, [1.0] * 9, 1, "speedup", 2.0, 0)
    with pytest.raises(ValueError):
        dy.dybit_search_bitwidths([1.0] * 9, [1.0] * 8, 1, "speedup", 2.0, 1)
