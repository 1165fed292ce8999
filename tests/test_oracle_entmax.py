"""Pins for the oracle's alpha-entmax (Eq. 2) against facts the paper and the mathematics fix."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.optimize import minimize
from scipy.special import softmax

from oracle import dash_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "entmax_closed_forms.txt")


def _rows():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            a, s1, s2, p1, p2 = map(float, line.split())
            out.append((a, s1, s2, p1, p2))
    return out


@pytest.mark.parametrize("alpha,s1,s2,p1,p2", _rows())
def test_hand_derived_two_element_values(alpha, s1, s2, p1, p2):
    p = orc.entmax(np.array([s1, s2]), alpha)
    assert np.allclose(p, [p1, p2], atol=1e-13)


def test_hand_derived_three_element_sparsemax():
    p = orc.entmax(np.array([1.0, 0.8, 0.1]), 2.0)
    assert np.allclose(p, [0.6, 0.4, 0.0], atol=1e-14)


def _brute_force_threshold(x, e):
    """Enumerate supports: S is the support iff the root tau_S of sum_S (x - tau)^e = 1
    satisfies x_i > tau_S on S and x_i <= tau_S off S.  Exactly one subset qualifies."""
    n = len(x)
    found = []
    for k in range(1, n + 1):
        for S in itertools.combinations(range(n), k):
            xs = x[list(S)]
            lo, hi = xs.min() - 1.0, xs.min()     # need tau < min_S x; f(min-1) >= 1 >= f(min)... bracket by growth
            # f_S(tau) = sum (xs - tau)^e - 1 is decreasing in tau on tau < min xs; may have no root there
            f = lambda t: np.sum((xs - t) ** e) - 1.0
            if f(hi) > 0:          # even at tau = min xs the sum exceeds 1: no root with all of S positive
                continue
            while f(lo) < 0:
                lo -= 1.0
            for _ in range(200):
                mid = 0.5 * (lo + hi)
                if f(mid) >= 0:
                    lo = mid
                else:
                    hi = mid
            tau = 0.5 * (lo + hi)
            off = np.delete(x, list(S))
            if np.all(xs > tau) and np.all(off <= tau):
                found.append((S, tau))
    return found


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.75])
def test_threshold_against_support_enumeration(alpha):
    rng = np.random.default_rng(7)
    e = 1.0 / (alpha - 1.0)
    for trial in range(12):
        n = int(rng.integers(2, 7))
        x = rng.normal(size=n) * rng.choice([0.2, 1.0, 3.0])
        found = _brute_force_threshold(x, e)
        assert len(found) == 1, (x, found)
        S, tau = found[0]
        t = orc.entmax_threshold(x, alpha)
        assert abs(t - tau) < 1e-10
        assert set(np.nonzero(x > t)[0]) == set(S)


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_simplex_and_zero_pattern(alpha):
    rng = np.random.default_rng(1)
    for n in (1, 2, 5, 33, 257, 2047):
        s = rng.normal(size=n) * 3.0
        p = orc.entmax(s, alpha)
        assert np.all(p >= 0)
        assert abs(p.sum() - 1.0) < 1e-11
        tau = orc.entmax_threshold((alpha - 1) * s, alpha)
        assert np.array_equal(p == 0, (alpha - 1) * s <= tau)


def test_alpha2_is_euclidean_projection_onto_simplex():
    """alpha = 2 is sparsemax = argmin_p ||s - p||_2 over the simplex: compare with a generic
    constrained solver and check no feasible point is closer."""
    rng = np.random.default_rng(3)
    for n in (3, 6, 10):
        s = rng.normal(size=n)
        p = orc.entmax(s, 2.0)
        res = minimize(lambda q: np.sum((q - s) ** 2), np.full(n, 1.0 / n), method="SLSQP",
                       bounds=[(0, 1)] * n, constraints=[{"type": "eq", "fun": lambda q: q.sum() - 1}],
                       options={"ftol": 1e-14, "maxiter": 500})
        assert np.allclose(res.x, p, atol=1e-6)
        for _ in range(200):
            q = rng.dirichlet(np.ones(n))
            assert np.sum((q - s) ** 2) >= np.sum((p - s) ** 2) - 1e-12


@pytest.mark.parametrize("alpha", [1.25, 1.5])
def test_maximises_tsallis_regularised_objective(alpha):
    """entmax(z) = argmax_p p.z + H_alpha(p), H_alpha = sum (p - p^alpha) / (alpha (alpha-1))."""
    rng = np.random.default_rng(5)

    def obj(p, z):
        return p @ z + np.sum(p - p ** alpha) / (alpha * (alpha - 1.0))

    for n in (4, 9):
        z = rng.normal(size=n) * 2.0
        p = orc.entmax(z, alpha)
        best = obj(p, z)
        for _ in range(300):
            q = rng.dirichlet(np.ones(n) * rng.choice([0.3, 1.0, 5.0]))
            assert obj(q, z) <= best + 1e-12
        res = minimize(lambda q: -obj(np.clip(q, 0, 1), z), np.full(n, 1.0 / n), method="SLSQP",
                       bounds=[(0, 1)] * n, constraints=[{"type": "eq", "fun": lambda q: q.sum() - 1}],
                       options={"ftol": 1e-14, "maxiter": 500})
        assert np.allclose(res.x, p, atol=2e-5)


def test_alpha_to_one_tends_to_softmax():
    rng = np.random.default_rng(11)
    s = rng.normal(size=40)
    ref = softmax(s)
    errs = [np.abs(orc.entmax(s, 1.0 + eps) - ref).max() for eps in (0.1, 0.03, 0.01, 0.003)]
    assert all(errs[i + 1] < errs[i] for i in range(len(errs) - 1))
    assert errs[-1] < 2e-3


def test_support_shrinks_with_alpha_and_shift_invariance():
    rng = np.random.default_rng(13)
    for _ in range(10):
        s = rng.normal(size=200) * 2.0
        sizes = [(orc.entmax(s, a) > 0).sum() for a in (1.25, 1.5, 2.0)]
        assert sizes[0] >= sizes[1] >= sizes[2] >= 1
        for a in (1.25, 1.5, 2.0):
            assert np.allclose(orc.entmax(s, a), orc.entmax(s + 17.25, a), atol=1e-12)


@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_sort_based_and_bisection_agree(alpha):
    rng = np.random.default_rng(17)
    for n in (1, 2, 3, 64, 1000, 2047):
        x = rng.normal(size=n) * rng.choice([0.01, 1.0, 5.0])
        assert abs(orc.entmax_threshold(x, alpha) - orc.entmax_threshold_bisect(x, alpha)) < 1e-11


def test_equal_scores_get_equal_weight():
    for alpha in (1.25, 1.5, 2.0):
        p = orc.entmax(np.array([0.3, 0.3, 0.3, -5.0]), alpha)
        assert np.allclose(p[:3], 1.0 / 3.0) and p[3] == 0.0
        assert np.allclose(orc.entmax(np.zeros(7), alpha), 1.0 / 7.0)


def test_rejects_bad_inputs():
    with pytest.raises(ValueError):
        orc.entmax(np.array([1.0]), 1.0)
    with pytest.raises(ValueError):
        orc.entmax_threshold(np.zeros(0), 1.5)
