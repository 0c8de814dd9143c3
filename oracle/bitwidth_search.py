"""Layer-wise bitwidth search (Section III-C.3, Algorithm 1; Eq. 3 and Eq. 4) -- test infrastructure, not a
product path.  Only tests/ and the benchmark's CPU legs may import this file.

The search is written here as a walk over an explicit "schedule" of single moves.  A move lowers ONE operand
(weights or activations) of ONE layer by one level, 8 -> 4 or 4 -> 2.  Every round of the search

  1. reads the current per-layer latency and error (they depend on the layers' current bitwidths),
  2. picks k candidate layers and orders them (by the strategy's two keys),
  3. lays the moves out as: weights of the candidates in that order, then activations in the same order,
  4. plays the moves one at a time, re-evaluating the whole-model total after each, and stops the whole
     search at the first move after which the strategy's stopping rule holds.

Strategy "speedup" (Eq. 3): candidates = the k slowest layers, ordered by ascending error; stop as soon as
alpha * total latency <= total latency at (8, 8).
Strategy "rmse" (Eq. 4): candidates = the k layers with the least error, ordered by descending latency; the total
error may never exceed beta * total error at (8, 8).

Readings where the paper is silent (each one is pinned by a hand-traced case in tests/test_bitwidth_search.py):
  * Eq. 4 is a budget: the first move that would push the total error above it is not taken, and the search ends
    there (the model returned always satisfies Eq. 4).
  * An operand already at 2 bits has no move; a layer with both operands at 2 bits is not a candidate.
  * Equal keys are ordered by layer index.
  * A round in which no move exists ends the search (everything is at 2 bits).

Tables are arrays of shape [N, 3, 3]: layer, activation level, weight level, with level 0 / 1 / 2 = 8 / 4 / 2 bits.
"""
from __future__ import annotations

import numpy as np

BITS_OF_LEVEL = (8, 4, 2)
LOWEST = len(BITS_OF_LEVEL) - 1


def as_table(per_layer_dicts) -> np.ndarray:
    """[{(a_bits, w_bits): value}] -> array [N, 3, 3] indexed by level."""
    t = np.empty((len(per_layer_dicts), 3, 3), dtype=np.float64)
    for i, d in enumerate(per_layer_dicts):
        for ia, a in enumerate(BITS_OF_LEVEL):
            for iw, w in enumerate(BITS_OF_LEVEL):
                t[i, ia, iw] = d[(a, w)]
    return t


class _Model:
    """Current level of every layer's activations and weights, and the tables they index."""

    def __init__(self, lat: np.ndarray, err: np.ndarray):
        self.lat, self.err = lat, err
        self.n = lat.shape[0]
        self.level = {"W": np.zeros(self.n, dtype=int), "A": np.zeros(self.n, dtype=int)}
        self.rows = np.arange(self.n)

    def per_layer(self, table):
        return table[self.rows, self.level["A"], self.level["W"]]

    def total(self, table) -> float:
        # summed in layer order, one addition per layer
        s = 0.0
        for v in self.per_layer(table):
            s += float(v)
        return s

    def bits(self, operand):
        return [BITS_OF_LEVEL[v] for v in self.level[operand]]


def _candidates(model: _Model, strategy: str, k: int):
    lat_now, err_now = model.per_layer(model.lat), model.per_layer(model.err)
    movable = [i for i in range(model.n) if model.level["W"][i] < LOWEST or model.level["A"][i] < LOWEST]
    if strategy == "speedup":
        first_key = {i: (-lat_now[i], i) for i in movable}         # slowest first
        second_key = {i: (err_now[i], i) for i in movable}         # then least error first
    else:
        first_key = {i: (err_now[i], i) for i in movable}          # least error first
        second_key = {i: (-lat_now[i], i) for i in movable}        # then slowest first
    chosen = sorted(movable, key=first_key.get)[:k]
    return sorted(chosen, key=second_key.get)


def search(lat, rmse, strategy: str, constraint: float, k: int, trace: list | None = None):
    """lat, rmse: arrays [N, 3, 3] (or lists of {(a_bits, w_bits): value} dicts).  Returns (W, A) as lists of
    bitwidths.  `trace`, if given, receives one (layer, operand, new_bits, total_after) tuple per move taken."""
    if strategy not in ("speedup", "rmse"):
        raise ValueError(strategy)
    lat = lat if isinstance(lat, np.ndarray) else as_table(lat)
    rmse = rmse if isinstance(rmse, np.ndarray) else as_table(rmse)
    model = _Model(lat, rmse)
    watched = lat if strategy == "speedup" else rmse
    reference = model.total(watched)                                # the (8, 8) model

    if strategy == "speedup" and constraint * reference <= reference:
        return model.bits("W"), model.bits("A")                     # alpha <= 1: nothing to do

    while True:
        order = _candidates(model, strategy, k)
        schedule = [(i, "W") for i in order] + [(i, "A") for i in order]
        moved = False
        for layer, operand in schedule:
            lv = model.level[operand]
            if lv[layer] == LOWEST:
                continue
            lv[layer] += 1
            after = model.total(watched)
            if strategy == "rmse" and after > constraint * reference:
                lv[layer] -= 1                                      # over the Eq. 4 budget: not taken, search over
                return model.bits("W"), model.bits("A")
            moved = True
            if trace is not None:
                trace.append((layer, operand, BITS_OF_LEVEL[lv[layer]], after))
            if strategy == "speedup" and constraint * after <= reference:
                return model.bits("W"), model.bits("A")             # Eq. 3 holds
        if not moved:
            return model.bits("W"), model.bits("A")                 # every operand is at 2 bits
