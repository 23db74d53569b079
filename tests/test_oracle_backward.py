"""Pins for the CPU oracle's backward (Eq. 5 of the paper)."""
import os

import numpy as np
import pytest

from oracle import lapsum_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gradcheck_table.txt")


def sigma(u):
    return np.where(u <= 0, 0.5 * np.exp(np.minimum(u, 0)), 1 - 0.5 * np.exp(-np.maximum(u, 0)))


def p_of(r64, k, t):
    """mask for fp64 scores: threshold from the oracle's sorted solve, CDF by numpy"""
    b = O.solve_sorted(np.sort(r64), k, t).b
    return sigma((r64 - b) / t), b


def fd_vjp(r64, v64, k, t, eps=1e-5):
    g = np.empty_like(r64)
    for j in range(r64.shape[0]):
        rp, rm = r64.copy(), r64.copy()
        rp[j] += eps
        rm[j] -= eps
        g[j] = (np.dot(v64, p_of(rp, k, t)[0]) - np.dot(v64, p_of(rm, k, t)[0])) / (2 * eps)
    return g


def golden_rows():
    rows = []
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            B, n, k, alpha, abs_err, rel_err = line.split()
            rows.append((int(B), int(n), float(k), float(alpha), float(abs_err), float(rel_err)))
    return rows


@pytest.mark.parametrize("B,n,k,alpha,abs_err,rel_err", golden_rows())
def test_vjp_matches_centred_finite_differences(B, n, k, alpha, abs_err, rel_err):
    # the paper's recipe: centred FD, eps = 1e-5, fp64, rel err = max abs err / max|g_FD|,
    # pass threshold 1e-3; the paper prints 4e-11 .. 3e-10 at these shapes
    rng = np.random.default_rng(100 + n + int(k))
    worst = 0.0
    for _ in range(B):
        r = rng.standard_normal(n).astype(np.float32)
        v = rng.standard_normal(n).astype(np.float32)
        b = O.forward(r, k, alpha).b[0]
        g = O.backward(v, r, b, alpha)[0]
        g_fd = fd_vjp(r.astype(np.float64), v.astype(np.float64), k, -alpha)
        worst = max(worst, float(np.max(np.abs(g - g_fd)) / np.max(np.abs(g_fd))))
    assert worst < 1e-3          # the paper's pass threshold
    assert worst < 1e-7          # same order as the printed 1e-10 level (FD truncation bounds it)
    assert rel_err < 1e-3        # the fixture itself is a pass row


def test_shift_invariance_sum_of_grad_is_zero():
    rng = np.random.default_rng(1)
    for n, k, t in [(64, 8.0, 0.5), (500, 33.3, 0.05), (2000, 100.0, 1.0)]:
        r = rng.standard_normal(n).astype(np.float32)
        v = rng.standard_normal(n).astype(np.float32)
        b = O.forward(r, k, -t).b[0]
        g = O.backward(v, r, b, -t)[0]
        assert abs(g.sum()) <= 1e-12 * np.abs(g).sum() + 1e-300


def test_constant_upstream_gives_zero_gradient():
    rng = np.random.default_rng(2)
    r = rng.standard_normal(100).astype(np.float32)
    b = O.forward(r, 10.0, -0.3).b[0]
    g = O.backward(np.ones(100, np.float32), r, b, -0.3)[0]
    assert np.max(np.abs(g)) <= 1e-15


def test_jacobian_is_symmetric():
    # J = diag(f) - f f^T / sum f, so e_i^T J e_j = e_j^T J e_i
    rng = np.random.default_rng(3)
    n = 24
    r = rng.standard_normal(n).astype(np.float32)
    b = O.forward(r, 5.0, -0.4).b[0]
    J = np.stack([O.backward(np.eye(n, dtype=np.float32)[i], r, b, -0.4)[0] for i in range(n)])
    assert np.allclose(J, J.T, atol=1e-15)
    # and it matches the closed form with f = min(p, 1-p)/t
    p = O.forward(r, 5.0, -0.4).p[0]
    f = np.minimum(p, 1 - p) / 0.4
    assert np.allclose(J, np.diag(f) - np.outer(f, f) / f.sum(), atol=1e-13)


def test_equal_scores_gradient_is_centred_upstream():
    n, k, t = 32, 8.0, 0.7
    r = np.full(n, 1.25, np.float32)
    v = np.random.default_rng(4).standard_normal(n).astype(np.float32)
    b = O.forward(r, k, -t).b[0]
    g = O.backward(v, r, b, -t)[0]
    f = np.exp(-abs(b - 1.25) / t) / (2 * t)
    assert np.allclose(g, f * (v.astype(np.float64) - v.astype(np.float64).mean()), atol=1e-14)


def test_underflowing_density_gives_zero_gradient():
    r = np.array([0.0, 1000.0], np.float32)
    g = O.backward(np.array([1.0, -1.0], np.float32), r, 500.0, -0.1)
    assert np.all(g == 0.0)


def loss_of(r64, v64, k, t):
    return float(np.dot(v64, p_of(r64, k, t)[0]))


@pytest.mark.parametrize("n,k,alpha", [(32, 4.0, -1.0), (64, 8.5, -0.5), (64, 16.0, -2.0), (200, 33.3, -0.1)])
def test_scalar_gradients_match_finite_differences(n, k, alpha):
    # the paper's applications learn k and alpha; it prints no formula, so the derived ones are pinned by
    # centred differences of L = <v, p> in fp64 (same recipe as the gradcheck table: eps = 1e-5)
    rng = np.random.default_rng(900 + n)
    r = rng.standard_normal(n).astype(np.float32)
    v = rng.standard_normal(n).astype(np.float32)
    r64, v64, t = r.astype(np.float64), v.astype(np.float64), -alpha
    b = O.forward(r, k, alpha).b[0]
    gk, ga = O.backward_scalars(v, r, b, alpha)
    eps = 1e-5
    fd_k = (loss_of(r64, v64, k + eps, t) - loss_of(r64, v64, k - eps, t)) / (2 * eps)
    fd_a = (loss_of(r64, v64, k, -(alpha + eps)) - loss_of(r64, v64, k, -(alpha - eps))) / (2 * eps)
    assert gk[0] == pytest.approx(fd_k, rel=1e-6, abs=1e-9)
    assert ga[0] == pytest.approx(fd_a, rel=1e-6, abs=1e-9)


def test_scalar_gradients_special_cases():
    rng = np.random.default_rng(5)
    r = rng.standard_normal(50).astype(np.float32)
    b = O.forward(r, 7.0, -0.3).b[0]
    # constant upstream: L = c * sum p = c * k, so dL/dk = c and dL/dalpha = 0
    gk, ga = O.backward_scalars(np.full(50, 2.5, np.float32), r, b, -0.3)
    assert gk[0] == pytest.approx(2.5, rel=1e-13) and abs(ga[0]) < 1e-12
    # dp/dk sums to one: with v = e_i the k-gradients over i add up to 1
    tot = sum(O.backward_scalars(np.eye(50, dtype=np.float32)[i], r, b, -0.3)[0][0] for i in range(50))
    assert tot == pytest.approx(1.0, rel=1e-12)
