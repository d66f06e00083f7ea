"""Pins of the bit-width assignment oracle (Section IV-A, Algorithm 1): hand-worked values, closed forms and
the invariants the algorithm is known to have, none of them computed by the code under test."""
import itertools
import math

import numpy as np
import pytest

from oracle import assign as A


def _rand_problem(seed, n=24, c=4, p=1):
    rng = np.random.default_rng(seed)
    X = rng.random((n, p)).tolist()
    U0 = rng.random((n, c)) + 0.05
    U0 = (U0 / U0.sum(axis=1, keepdims=True)).tolist()
    return X, U0


def test_hand_worked_two_points_one_iteration():
    # X = {0, 1}, U0 = [[.8,.2],[.2,.8]], m = 2:
    #   v_1 = (0.64*0 + 0.04*1)/0.68 = 1/17, v_2 = 16/17
    #   u_11 = 1/(1 + ((1/17)/(16/17))^2) = 256/257, u_12 = 1/257, and mirrored for x_2
    V, U, it, _ = A.fuzzy_cmeans([[0.0], [1.0]], [[0.8, 0.2], [0.2, 0.8]], m=2.0, eps=1e-30, max_iter=1)
    assert it == 1
    assert V[0][0] == pytest.approx(1 / 17, abs=1e-15) and V[1][0] == pytest.approx(16 / 17, abs=1e-15)
    assert U[0][0] == pytest.approx(256 / 257, abs=1e-15) and U[0][1] == pytest.approx(1 / 257, abs=1e-15)
    assert U[1][1] == pytest.approx(256 / 257, abs=1e-15) and U[1][0] == pytest.approx(1 / 257, abs=1e-15)


def test_hand_worked_fuzzifier_three():
    # m = 3: exponent 2/(m-1) = 1, weights u^3.  X = {0, 2}, U0 = [[.5,.5],[.25,.75]]
    #   v_1 = (0.015625*2)/(0.125+0.015625) = 2/9,  v_2 = (0.421875*2)/(0.125+0.421875) = 54/35
    #   x_1 = 0: d = (2/9, 54/35): u_11 = 1/(1 + (2/9)/(54/35)) = 243/278
    V, U, _, _ = A.fuzzy_cmeans([[0.0], [2.0]], [[0.5, 0.5], [0.25, 0.75]], m=3.0, eps=1e-30, max_iter=1)
    assert V[0][0] == pytest.approx(2 / 9, abs=1e-15) and V[1][0] == pytest.approx(54 / 35, abs=1e-15)
    assert U[0][0] == pytest.approx(243 / 278, abs=1e-15)
    d1, d2 = 2 - 2 / 9, 2 - 54 / 35
    assert U[1][1] == pytest.approx(1 / (1 + d2 / d1), abs=1e-15)


def test_single_cluster_is_the_mean():
    X, _ = _rand_problem(1, n=10, c=1, p=3)
    V, U, it, _ = A.fuzzy_cmeans(X, [[1.0]] * 10, m=2.0)
    assert np.allclose(V[0], np.mean(np.array(X), axis=0), rtol=0, atol=1e-15)
    assert all(r == [1.0] for r in U)


@pytest.mark.parametrize("m", [1.5, 2.0, 3.0])
def test_rows_stochastic_objective_descends_and_fixed_point(m):
    X, U0 = _rand_problem(7, n=30, c=4, p=2)
    V, U, it, hist = A.fuzzy_cmeans(X, U0, m=m, eps=1e-12, max_iter=5000)
    Un = np.array(U)
    assert np.all(Un >= 0) and np.all(Un <= 1) and np.allclose(Un.sum(axis=1), 1.0, atol=1e-14)
    # Bezdek: both half-steps minimise J_m in their block of variables, so J_m never rises
    assert all(b <= a * (1 + 1e-13) for a, b in zip(hist, hist[1:]))
    assert it < 5000
    # at convergence the centers are the u^m-weighted means of the returned U (independent numpy form)
    W = Un ** m
    assert np.allclose(np.array(V), (W.T @ np.array(X)) / W.sum(axis=0)[:, None], atol=1e-9)
    # and each row of U satisfies the stationarity condition in its inverse-distance form
    D = np.linalg.norm(np.array(X)[:, None, :] - np.array(V)[None, :, :], axis=2)
    R = D ** (-2.0 / (m - 1.0))
    assert np.allclose(Un, R / R.sum(axis=1, keepdims=True), atol=1e-12)


def test_membership_update_minimises_objective_bruteforce():
    # for fixed centers, the update's row must beat every other row of the simplex (grid search, n = 1, c = 3)
    x, V, m = [[0.3]], [[0.0], [0.5], [1.0]], 2.0
    u = A.memberships(x, V, m)[0]
    best = A.objective(x, [u], V, m)
    grid = np.linspace(0, 1, 101)
    for a, b in itertools.product(grid, grid):
        if a + b <= 1.0:
            assert A.objective(x, [[a, b, 1 - a - b]], V, m) >= best - 1e-15


def test_separated_groups_are_recovered():
    rng = np.random.default_rng(3)
    means = [0.0, 10.0, 20.0, 30.0]
    labels = rng.integers(0, 4, 40)
    labels[:4] = [0, 1, 2, 3]
    X = [[means[l] + 0.01 * rng.standard_normal()] for l in labels]
    U0 = A.initial_memberships([v[0] for v in X], 4, 2.0)
    V, U, _, _ = A.fuzzy_cmeans(X, U0, m=2.0, eps=1e-12)
    got = sorted(v[0] for v in V)
    assert np.allclose(got, means, atol=0.02)
    bits, hard = A.assign_bits(V, U, [8, 4, 3, 2])
    assert bits == [[2, 3, 4, 8][l] for l in labels]
    assert min(max(r) for r in U) > 0.999


def test_points_on_the_centers_are_one_hot():
    X = [[1.0], [5.0], [5.0], [1.0], [9.0]]
    U = A.memberships(X, [[1.0], [5.0], [9.0]], 2.0)
    assert U == [[1, 0, 0], [0, 1, 0], [0, 1, 0], [1, 0, 0], [0, 0, 1]]
    U = A.memberships([[2.0]], [[2.0], [2.0], [7.0]], 2.0)
    assert U == [[0.5, 0.5, 0.0]]
    # one-hot memberships on distinct values are a fixed point: centers = the values
    V, U2, it, _ = A.fuzzy_cmeans(X, [[1, 0, 0], [0, 1, 0], [0, 1, 0], [1, 0, 0], [0, 0, 1]], m=2.0)
    assert V == [[1.0], [5.0], [9.0]] and it == 1


def test_equivariance_under_relabelling_and_affine_maps():
    X, U0 = _rand_problem(11, n=16, c=3, p=1)
    V, U, it, _ = A.fuzzy_cmeans(X, U0, m=2.0, eps=1e-13, max_iter=3000)
    perm = [2, 0, 1]
    Vp, Up, itp, _ = A.fuzzy_cmeans(X, [[r[k] for k in perm] for r in U0], m=2.0, eps=1e-13, max_iter=3000)
    assert itp == it
    assert np.allclose(np.array(Vp), np.array(V)[perm], atol=1e-12)
    assert np.allclose(np.array(Up), np.array(U)[:, perm], atol=1e-12)
    rows = list(reversed(range(16)))
    Vr, Ur, _, _ = A.fuzzy_cmeans([X[i] for i in rows], [U0[i] for i in rows], m=2.0, eps=1e-13, max_iter=3000)
    assert np.allclose(np.array(Vr), np.array(V), atol=1e-10) and np.allclose(np.array(Ur), np.array(U)[rows], atol=1e-10)
    Xa = [[4.0 * v[0] - 3.0] for v in X]                    # exact in binary floating point up to rounding
    Va, Ua, _, _ = A.fuzzy_cmeans(Xa, U0, m=2.0, eps=1e-13, max_iter=3000)
    assert np.allclose(np.array(Va), 4.0 * np.array(V) - 3.0, atol=1e-9) and np.allclose(np.array(Ua), np.array(U), atol=1e-9)


def test_initial_memberships_from_shares():
    share = [0.05, 0.10, 0.25, 0.60]
    U0 = A.initial_memberships(share, 4, 2.0)
    assert np.allclose(np.sum(U0, axis=1), 1.0, atol=1e-15)
    # anchors at 0.05, 0.2333.., 0.4166.., 0.60: the extreme shares sit on the outer anchors
    assert U0[0] == [1.0, 0.0, 0.0, 0.0] and U0[3] == [0.0, 0.0, 0.0, 1.0]
    # share 0.10 against the anchors, inverse-square weights by hand
    anchors = [0.05 + 0.55 * k / 3 for k in range(4)]
    w = [1 / (0.10 - a) ** 2 for a in anchors]
    assert np.allclose(U0[1], [v / sum(w) for v in w], atol=1e-14)
    assert A.initial_memberships([0.25] * 4, 4) == [[0.25] * 4] * 4


def test_precision_map_and_low_precision_first():
    V = [[0.2], [0.9], [0.5], [0.05]]                       # significance order of the clusters: 1, 2, 0, 3
    U = [[0.7, 0.1, 0.1, 0.1],                              # cluster 0 -> third level
         [0.05, 0.8, 0.1, 0.05],                            # cluster 1 -> highest
         [0.1, 0.42, 0.40, 0.08],                           # clusters 1 and 2 overlap
         [0.0, 0.0, 0.1, 0.9],                              # cluster 3 -> lowest
         [0.25, 0.25, 0.25, 0.25]]                          # exact tie -> lowest precision of the tied
    assert A.cluster_order(V, U) == [1, 2, 0, 3]
    bits, hard = A.assign_bits(V, U, [8, 6, 4, 2], overlap=0.0)
    assert bits == [4, 8, 8, 2, 2] and hard == [0, 1, 1, 3, 3]
    bits, hard = A.assign_bits(V, U, [8, 6, 4, 2], overlap=0.05)
    assert bits == [4, 8, 6, 2, 2] and hard == [0, 1, 2, 3, 3]
    # overlap between a lower (largest membership) and a higher cluster keeps the lower one
    bits, _ = A.assign_bits(V, [[0.1, 0.40, 0.42, 0.08]], [8, 6, 4, 2], overlap=0.05)
    assert bits == [6]
    # equal centers: the larger membership mass ranks first, then the lower index
    assert A.cluster_order([[0.5], [0.5], [0.5]], [[0.2, 0.5, 0.3], [0.2, 0.5, 0.3]]) == [1, 2, 0]
