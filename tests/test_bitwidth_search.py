"""Algorithm 1 (Section III-C.3): the oracle's search against hand-traced runs, against brute force over all
(3 x 3)^N assignments on tiny models, and the library's host implementation against the oracle on random tables.

The hand-traced cases use tables a reader can evaluate in the head:
    Lat_i(a, w)  = L_i * (a + w) / 16          (8,8) -> L_i, (8,4)/(4,8) -> 0.75 L_i, (4,4) -> 0.5 L_i, ... (2,2) -> 0.25 L_i
    RMSE_i(a, w) = R_i * (g(a) + g(w)),  g(8) = 1, g(4) = 2, g(2) = 4        (8,8) -> 2 R_i
Each expected result is worked out in the comment above it from Algorithm 1 and Eq. 3 / Eq. 4, not from a run.
"""
import itertools

import numpy as np
import pytest

import paper_2302_12510_b200 as dy
from oracle import bitwidth_search as bs

LEVELS = (8, 4, 2)
G = {8: 1.0, 4: 2.0, 2: 4.0}


def _simple(Ls, Rs):
    lat = [{(a, w): L * (a + w) / 16.0 for a in LEVELS for w in LEVELS} for L in Ls]
    rmse = [{(a, w): R * (G[a] + G[w]) for a in LEVELS for w in LEVELS} for R in Rs]
    return lat, rmse


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


def test_hand_traced_speedup_k1():
    # L = (8, 2), alpha = 2: base 10, goal total <= 5.  Round 1: slowest = layer 0.  W0 8->4: 6 + 2 = 8, no.
    # A0 8->4: 4 + 2 = 6, no.  Round 2: latencies (4, 2), slowest still layer 0.  W0 4->2: 3 + 2 = 5 <= 5: stop.
    lat, rmse = _simple([8.0, 2.0], [0.01, 0.10])
    trace = []
    assert bs.search(lat, rmse, "speedup", 2.0, 1, trace) == ([2, 8], [4, 8])
    assert [(t[0], t[1], t[2]) for t in trace] == [(0, "W", 4), (0, "A", 4), (0, "W", 2)]
    assert [t[3] for t in trace] == [8.0, 6.0, 5.0]


def test_hand_traced_speedup_k2_second_candidate_moves_before_the_goal_is_met():
    # L = (8, 6, 1), R = (3, 1, 2), k = 2, alpha = 1.4: base 15, goal total <= 10.714.
    # Lat_rank: the two slowest are layers 0 and 1; RMSE_rerank puts layer 1 (2 R = 2) before layer 0 (6).
    # W1 8->4: 8 + 4.5 + 1 = 13.5, no.  W0 8->4: 6 + 4.5 + 1 = 11.5, no.  A1 8->4: 6 + 3 + 1 = 10 <= 10.714: stop.
    lat, rmse = _simple([8.0, 6.0, 1.0], [3.0, 1.0, 2.0])
    trace = []
    assert bs.search(lat, rmse, "speedup", 1.4, 2, trace) == ([4, 4, 8], [8, 4, 8])
    assert [(t[0], t[1]) for t in trace] == [(1, "W"), (0, "W"), (1, "A")]
    # (descending-error order would give A = [4, 8, 8]; k taken as 1 would give W = [4, 4, 8], A = [4, 8, 8])


def test_hand_traced_speedup_ranking_is_recomputed_every_round():
    # L = (8, 6, 1), k = 1, alpha = 1.6: goal total <= 9.375.  Round 1: layer 0.  W0: 6 + 6 + 1 = 13; A0: 4 + 6 + 1 = 11.
    # Round 2: latencies are now (4, 6, 1), so the slowest is layer 1.  W1: 4 + 4.5 + 1 = 9.5, no;
    # A1: 4 + 3 + 1 = 8 <= 9.375: stop.  (A ranking kept from round 1 would end at W = A = [2, 8, 8].)
    lat, rmse = _simple([8.0, 6.0, 1.0], [3.0, 1.0, 2.0])
    assert bs.search(lat, rmse, "speedup", 1.6, 1) == ([4, 4, 8], [4, 4, 8])


def test_hand_traced_rmse_rank_and_rerank_disagree_and_the_budget_takes_a_move_back():
    # L = (1, 10, 20), R = (1, 2, 3), k = 2, beta = 1.2: base error 2 * 6 = 12, budget 14.4.
    # RMSE_rank: the two least-error layers are 0 (2) and 1 (4) -- NOT the slow layer 2; Lat_rerank: layer 1
    # (latency 10) before layer 0 (1).  W1 8->4: error 2 + 6 + 6 = 14 <= 14.4, taken.  W0 8->4: 3 + 6 + 6 = 15 > 14.4:
    # not taken, search over.  (Ranking by latency would touch layer 2 first: 12 + 3 = 15 > 14.4, nothing changes;
    # re-ranking the other way round would lower layer 0 first and end at W = [4, 8, 8].)
    lat, rmse = _simple([1.0, 10.0, 20.0], [1.0, 2.0, 3.0])
    trace = []
    W, A = bs.search(lat, rmse, "rmse", 1.2, 2, trace)
    assert (W, A) == ([8, 4, 8], [8, 8, 8])
    assert trace == [(1, "W", 4, 14.0)]
    assert _tot(rmse, W, A) <= 1.2 * 12.0


def test_hand_traced_rmse_budget_exact_boundary_is_inside():
    # same model, beta = 1.25: budget 15 (all totals are small integers, so the comparison is exact).  W1: 14, taken;
    # W0: 15 <= 15, taken (the budget's edge is inside); then A1: 15 + 2 = 17 > 15: not taken, search over.
    lat, rmse = _simple([1.0, 10.0, 20.0], [1.0, 2.0, 3.0])
    assert bs.search(lat, rmse, "rmse", 1.25, 2) == ([4, 4, 8], [8, 8, 8])


def test_hand_traced_bottoms_out_at_2_2():
    # the fastest model is 4 x faster than (8, 8) with these tables, so alpha = 5 cannot be met: every operand ends
    # at 2 bits and the search returns instead of looping.  2 layers x 2 operands x 2 levels = 8 moves.
    lat, rmse = _simple([3.0, 5.0], [1.0, 1.0])
    trace = []
    assert bs.search(lat, rmse, "speedup", 5.0, 1, trace) == ([2, 2], [2, 2])
    assert len(trace) == 8
    # the error budget of Eq. 4 large enough for everything: same end state
    assert bs.search(lat, rmse, "rmse", 100.0, 2) == ([2, 2], [2, 2])


def test_alpha_not_above_one_changes_nothing():
    lat, rmse = _simple([3.0, 5.0], [1.0, 1.0])
    assert bs.search(lat, rmse, "speedup", 1.0, 2) == ([8, 8], [8, 8])


@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("n", [1, 2, 3])
def test_brute_force_feasibility_on_tiny_models(seed, n):
    """All 9^N assignments enumerated: Eq. 3 can be met iff the search meets it (latencies fall with the bits, so the
    search's last resort, all operands at 2 bits, is the fastest model); under Eq. 4 the search's answer is inside
    the budget and no slower than the (8, 8) model."""
    lat, rmse = _tables(n, 50 + seed)
    combos = list(itertools.product(LEVELS, repeat=2 * n))
    base_l, base_r = _tot(lat, [8] * n, [8] * n), _tot(rmse, [8] * n, [8] * n)
    best_l = min(_tot(lat, c[:n], c[n:]) for c in combos)
    for alpha in (1.3, 2.0, 4.0, 12.0, 40.0):
        W, A = bs.search(lat, rmse, "speedup", alpha, n)
        feasible = alpha * best_l <= base_l
        assert (alpha * _tot(lat, W, A) <= base_l) == feasible
        if not feasible:
            assert set(W) | set(A) == {2}
    for beta in (1.05, 1.5, 3.0, 8.0):
        W, A = bs.search(lat, rmse, "rmse", beta, n)
        assert _tot(rmse, W, A) <= beta * base_r
        assert _tot(lat, W, A) <= base_l


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


def _flat(t, n):
    return [t[i][(a, w)] for i in range(n) for a in LEVELS for w in LEVELS]


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("strategy,c,k", [("speedup", 2.5, 1), ("speedup", 5.0, 4), ("rmse", 1.8, 2), ("rmse", 4.0, 3)])
def test_library_search_equals_oracle(seed, strategy, c, k):
    n = 9
    lat, rmse = _tables(n, seed + 100)
    W, A = bs.search(lat, rmse, strategy, c, k)
    Wl, Al = dy.dybit_search_bitwidths(_flat(lat, n), _flat(rmse, n), n, strategy, c, k)
    assert (Wl, Al) == (W, A)


def test_library_search_on_the_hand_traced_cases():
    """The library's host code against the values worked out by hand above (not via the oracle)."""
    lat, rmse = _simple([8.0, 6.0, 1.0], [3.0, 1.0, 2.0])
    assert dy.dybit_search_bitwidths(_flat(lat, 3), _flat(rmse, 3), 3, "speedup", 1.4, 2) == ([4, 4, 8], [8, 4, 8])
    assert dy.dybit_search_bitwidths(_flat(lat, 3), _flat(rmse, 3), 3, "speedup", 1.6, 1) == ([4, 4, 8], [4, 4, 8])
    lat, rmse = _simple([1.0, 10.0, 20.0], [1.0, 2.0, 3.0])
    assert dy.dybit_search_bitwidths(_flat(lat, 3), _flat(rmse, 3), 3, "rmse", 1.2, 2) == ([8, 4, 8], [8, 8, 8])
    assert dy.dybit_search_bitwidths(_flat(lat, 3), _flat(rmse, 3), 3, "rmse", 1.25, 2) == ([4, 4, 8], [8, 8, 8])
    lat, rmse = _simple([3.0, 5.0], [1.0, 1.0])
    assert dy.dybit_search_bitwidths(_flat(lat, 2), _flat(rmse, 2), 2, "speedup", 5.0, 1) == ([2, 2], [2, 2])


def test_library_search_argument_errors():
    with pytest.raises(dy.DybitError):
        dy.dybit_search_bitwidths([1.0] * 9, [1.0] * 9, 1, "speedup", 2.0, 0)
    with pytest.raises(ValueError):
        dy.dybit_search_bitwidths([1.0] * 9, [1.0] * 8, 1, "speedup", 2.0, 1)
