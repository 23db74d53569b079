"""Pins for the CPU oracle with alpha > 0: Eq. 1 as printed, p_i = sigma((b - r_i)/alpha), which then selects the k
smallest scores.  None of these calls the code path they check in another guise: the bisection works on Eq. 1's sum
directly, the closed forms are worked by hand, the complement identity goes through the alpha < 0 solve, and the
gradients are checked by finite differences of the forward."""
import math

import numpy as np
import pytest

from oracle import lapsum_oracle as O


def sigma(u):
    return np.where(u <= 0, 0.5 * np.exp(np.minimum(u, 0)), 1 - 0.5 * np.exp(-np.maximum(u, 0)))


def cases():
    rng = np.random.default_rng(77)
    out = []
    for _ in range(30):
        n = int(rng.integers(2, 48))
        r = rng.standard_normal(n).astype(np.float32)
        if rng.random() < 0.3:
            r[rng.integers(0, n, n // 2)] = r[0]  # ties
        k = float(rng.uniform(0.2, n - 0.2)) if rng.random() < 0.5 else float(rng.integers(1, n))
        out.append((r, k, float(rng.choice([0.05, 0.3, 1.0, 4.0]))))
    return out


def test_forward_matches_bisection_on_eq1_itself():
    for r, k, alpha in cases():
        f = O.forward(r, k, alpha)
        p_bis = sigma((O.bisect(r, k, alpha) - r.astype(np.float64)) / alpha)
        assert np.max(np.abs(f.p[0] - p_bis)) <= 1e-12
        assert abs(f.p[0].sum() - k) <= 1e-11 * max(1.0, k)
        # the mask is Eq. 1 at the returned threshold
        assert np.max(np.abs(f.p[0] - sigma((f.b[0] - r.astype(np.float64)) / alpha))) <= 1e-15


def test_b_matches_bisection_when_well_conditioned():
    rng = np.random.default_rng(4)
    for _ in range(30):
        n = int(rng.integers(8, 64))
        r = rng.standard_normal(n).astype(np.float32)
        k = float(rng.uniform(0.5, n - 0.5))
        assert O.forward(r, k, 0.5).b[0] == pytest.approx(O.bisect(r, k, 0.5), abs=1e-11)


def test_single_score_closed_form():
    # n = 1: sigma((b - r)/alpha) = k  =>  b = r + alpha ln(2k) (k <= 1/2),  b = r - alpha ln(2(1-k)) (k > 1/2)
    for r0, k, a in [(0.3, 0.2, 0.7), (-1.5, 0.5, 0.1), (2.0, 0.9, 1.3)]:
        r = np.array([r0], np.float32)
        want = float(r[0]) + a * math.log(2 * k) if k <= 0.5 else float(r[0]) - a * math.log(2 * (1 - k))
        assert O.forward(r, k, a).b[0] == pytest.approx(want, abs=1e-13)


def test_mask_decreases_with_the_score_and_selects_the_smallest():
    rng = np.random.default_rng(9)
    r = rng.standard_normal(40).astype(np.float32)
    p = O.forward(r, 5.0, 1e-4).p[0]
    order = np.argsort(r, kind="stable")
    assert np.all(np.diff(O.forward(r, 5.0, 0.7).p[0][order]) <= 0)
    # alpha -> 0+: the hard bottom-5 indicator (Theorem 1 mirrored)
    hard = np.zeros(40)
    hard[order[:5]] = 1.0
    assert np.max(np.abs(p - hard)) < 1e-9


def test_complement_identity_through_the_negative_alpha_solve():
    # sigma(-u) = 1 - sigma(u): sum_i sigma((b - r_i)/alpha) = k  <=>  sum_i sigma((r_i - b)/alpha) = n - k,
    # so the alpha > 0 problem with budget k has the threshold of the alpha < 0 problem with budget n - k
    for r, k, alpha in cases():
        n = r.shape[0]
        f, g = O.forward(r, k, alpha), O.forward(r, n - k, -alpha)
        assert np.max(np.abs(f.p[0] - (1.0 - g.p[0]))) <= 1e-12
        gap_ok = (k != round(k))  # integer budgets may sit on a plateau where b is not unique to rounding
        if gap_ok:
            assert f.b[0] == pytest.approx(g.b[0], abs=1e-10)


def loss(r, v64, k, alpha):
    """<v, p> with fp32 scores r (the oracle's input type)"""
    return float(np.dot(v64, O.forward(r, k, alpha).p[0]))


@pytest.mark.parametrize("n,k,alpha", [(24, 4.0, 1.0), (48, 8.5, 0.5), (64, 16.0, 2.0)])
def test_gradients_match_finite_differences(n, k, alpha):
    rng = np.random.default_rng(300 + n)
    # scores on a 2^-10 grid so that +-eps = 2^-12 steps are exact in fp32
    r = (np.round(rng.standard_normal(n) * 1024) / 1024).astype(np.float32)
    v = rng.standard_normal(n).astype(np.float32)
    v64 = v.astype(np.float64)
    b = O.forward(r, k, alpha).b[0]
    g = O.backward(v, r, b, alpha)[0]
    eps = 2.0 ** -12
    fd = np.empty(n)
    for j in range(n):
        rp, rm = r.copy(), r.copy()
        rp[j] += np.float32(eps)
        rm[j] -= np.float32(eps)
        fd[j] = (loss(rp, v64, k, alpha) - loss(rm, v64, k, alpha)) / (2 * eps)
    assert np.max(np.abs(g - fd)) <= 2e-6 * max(1.0, np.max(np.abs(fd)))  # O(eps^2) truncation
    gk, ga = O.backward_scalars(v, r, b, alpha)
    e = 1e-5
    assert gk[0] == pytest.approx((loss(r, v64, k + e, alpha) - loss(r, v64, k - e, alpha)) / (2 * e), rel=1e-6, abs=1e-9)
    assert ga[0] == pytest.approx((loss(r, v64, k, alpha + e) - loss(r, v64, k, alpha - e)) / (2 * e), rel=1e-6, abs=1e-9)


def test_gradient_is_minus_the_negative_alpha_gradient_at_the_same_threshold():
    rng = np.random.default_rng(12)
    r = rng.standard_normal(30).astype(np.float32)
    v = rng.standard_normal(30).astype(np.float32)
    b = O.forward(r, 7.5, 0.4).b[0]
    assert np.array_equal(O.backward(v, r, b, 0.4), -O.backward(v, r, b, -0.4))
    assert abs(O.backward(v, r, b, 0.4).sum()) < 1e-13  # shift invariance
