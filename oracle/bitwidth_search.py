"""Algorithm 1 (layer-wise bitwidth search), plain Python -- test infrastructure, not a product path.

Follows the paper's search flow step by step (Section III-C.3, Algorithm 1) with Eq. 3 / Eq. 4 as the stopping
rules.  Inputs are two tables per layer, indexed by (activation bits, weight bits) over {8, 4, 2}: latency
Lat_i(a, w) and error RMSE_i(a, w).  Readings where the paper is silent are stated next to the code.
"""
from __future__ import annotations

LEVELS = (8, 4, 2)


def _total(table, W, A):
    return sum(table[i][(A[i], W[i])] for i in range(len(W)))


def search(lat, rmse, strategy: str, constraint: float, k: int):
    """lat[i][(a, w)], rmse[i][(a, w)] for a, w in {8, 4, 2}.  strategy: "speedup" (Eq. 3, constraint = alpha)
    or "rmse" (Eq. 4, constraint = beta).  Returns (W, A) lists of bitwidths."""
    n = len(lat)
    W, A = [8] * n, [8] * n                                   # all layers start at (8, 8)
    total_table = lat if strategy == "speedup" else rmse
    base = _total(total_table, W, A)                          # metric_base

    def meets():
        cur = _total(total_table, W, A)
        if strategy == "speedup":
            return constraint * cur <= base                   # Eq. 3: alpha * sum Lat <= sum Lat(8,8)
        return cur > constraint * base                        # Eq. 4 budget used up (see degrade below)

    def degrade(layer_list, bits):
        """Degrade_level: one layer at a time, 8 -> 4 or 4 -> 2, stop as soon as the constraint is met."""
        changed = False
        for i in layer_list:
            if bits[i] == 2:
                continue
            old = bits[i]
            bits[i] = 4 if old == 8 else 2
            changed = True
            if strategy == "rmse" and _total(rmse, W, A) > constraint * base:
                bits[i] = old                                 # reading: Eq. 4 is a hard budget -> undo the step that breaks it
                return changed, True
            if meets():
                return changed, True
        return changed, False

    if meets() and strategy == "speedup":
        return W, A
    while True:
        lat_now = [lat[i][(A[i], W[i])] for i in range(n)]    # Layerwise_metric
        rmse_now = [rmse[i][(A[i], W[i])] for i in range(n)]
        live = [i for i in range(n) if W[i] > 2 or A[i] > 2]
        if not live:
            break
        if strategy == "speedup":
            top = sorted(live, key=lambda i: (-lat_now[i], i))[:k]          # Lat_rank: the k slowest layers
            order = sorted(top, key=lambda i: (rmse_now[i], i))             # RMSE_rerank: least error first
        else:
            top = sorted(live, key=lambda i: (rmse_now[i], i))[:k]          # RMSE_rank: the k least-error layers
            order = sorted(top, key=lambda i: (-lat_now[i], i))             # Lat_rerank: slowest first
        c1, done = degrade(order, W)
        if done:
            break
        c2, done = degrade(order, A)
        if done or not (c1 or c2):
            break
    return W, A
