"""CPU oracle of the offline bit-width assignment (Section IV-A, Algorithm 1).  TEST INFRASTRUCTURE ONLY.

Plain Python loops in float64, one statement per line of the algorithm, in the algorithm's order and notation:
X = {x_1..x_n} the synthesized expert significance (x_i a point of R^p, p = 1 in the paper), c clusters,
fuzzifier m > 1, tolerance eps, membership ("cluster score") matrix U [n][c], centers V [c][p].

Readings of what the paper leaves open (each is also an argument, so that a test can take another one):
  * ||U_new - U_old|| is the Frobenius norm.
  * A point that coincides with one or more centers shares its membership equally among those centers and has
    none elsewhere (the limit of the update formula).
  * The paper initialises U from each expert's share of the routed tokens, a scalar per expert while U has c
    columns: `initial_memberships` turns the shares into a row-stochastic matrix by one membership update
    against c anchors spread evenly from the smallest to the largest share.
  * The cluster of greatest significance takes the highest precision: clusters are ordered by the mean coordinate
    of their centers (ties: larger membership mass first, then lower cluster index).
  * Experts in the overlap of two clusters go to the lower precision: an expert whose two largest memberships
    differ by less than `overlap` takes the lower of the two clusters' precisions.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple


def _dist(a: Sequence[float], b: Sequence[float]) -> float:
    return math.sqrt(sum((u - v) * (u - v) for u, v in zip(a, b)))


def memberships(X: Sequence[Sequence[float]], V: Sequence[Sequence[float]], m: float) -> List[List[float]]:
    """u_ik = 1 / sum_j (||x_i - v_k|| / ||x_i - v_j||)^(2/(m-1))   (Algorithm 1, membership update)."""
    n, c = len(X), len(V)
    expo = 2.0 / (m - 1.0)
    U = [[0.0] * c for _ in range(n)]
    for i in range(n):
        d = [_dist(X[i], V[k]) for k in range(c)]
        zero = [k for k in range(c) if d[k] == 0.0]
        if zero:
            for k in zero:
                U[i][k] = 1.0 / len(zero)
            continue
        for k in range(c):
            U[i][k] = 1.0 / sum((d[k] / d[j]) ** expo for j in range(c))
    return U


def centers(X: Sequence[Sequence[float]], U: Sequence[Sequence[float]], m: float) -> List[List[float]]:
    """v_k = sum_i u_ik^m x_i / sum_i u_ik^m   (Algorithm 1, center update)."""
    n, c, p = len(X), len(U[0]), len(X[0])
    V = []
    for k in range(c):
        den = sum(U[i][k] ** m for i in range(n))
        V.append([sum(U[i][k] ** m * X[i][a] for i in range(n)) / den for a in range(p)])
    return V


def objective(X, U, V, m: float) -> float:
    """J_m = sum_i sum_k u_ik^m ||x_i - v_k||^2, the functional the two updates descend on."""
    return sum(U[i][k] ** m * _dist(X[i], V[k]) ** 2 for i in range(len(X)) for k in range(len(V)))


def fuzzy_cmeans(X, U0, m: float = 2.0, eps: float = 1e-9, max_iter: int = 1000):
    """Algorithm 1.  Returns (V, U, iterations, history) with history[t] = J_m after iteration t."""
    U = [list(r) for r in U0]
    hist = []
    it = 0
    while True:
        V = centers(X, U, m)
        U_new = memberships(X, V, m)
        it += 1
        hist.append(objective(X, U_new, V, m))
        diff = math.sqrt(sum((U_new[i][k] - U[i][k]) ** 2 for i in range(len(U)) for k in range(len(U[0]))))
        U = U_new
        if diff < eps or it >= max_iter:
            return V, U, it, hist


def initial_memberships(share: Sequence[float], c: int, m: float = 2.0) -> List[List[float]]:
    """Row-stochastic U from per-expert token shares: memberships of the share against c evenly spread anchors."""
    lo, hi = min(share), max(share)
    if c == 1 or hi == lo:
        return [[1.0 / c] * c for _ in share]
    anchors = [[lo + (hi - lo) * k / (c - 1)] for k in range(c)]
    return memberships([[s] for s in share], anchors, m)


def cluster_order(V, U) -> List[int]:
    """Clusters from the most to the least significant."""
    c = len(V)
    key = []
    for k in range(c):
        mean = sum(V[k]) / len(V[k])
        mass = sum(U[i][k] for i in range(len(U)))
        key.append((-mean, -mass, k))
    return [k for _, _, k in sorted(key)]


def assign_bits(V, U, levels: Sequence[int], overlap: float = 0.0) -> Tuple[List[int], List[int]]:
    """(bits per expert, cluster per expert).  levels[r] = precision of the r-th most significant cluster."""
    order = cluster_order(V, U)
    rank = {k: r for r, k in enumerate(order)}
    bits, hard = [], []
    for row in U:
        ks = sorted(range(len(row)), key=lambda k: (-row[k], -rank[k]))       # exact ties: the lower precision first
        k1 = ks[0]
        chosen = k1
        if len(ks) > 1 and row[ks[0]] - row[ks[1]] < overlap:
            k2 = ks[1]
            chosen = k1 if rank[k1] > rank[k2] else k2                          # the lower-precision cluster
        hard.append(chosen)
        bits.append(int(levels[rank[chosen]]))
    return bits, hard
