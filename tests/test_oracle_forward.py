"""Pins for the CPU oracle's forward (threshold b and mask p).

Every check here compares the oracle with something that is not the oracle:
the plain definition (full-sum bisection, brute-force node sums), closed
forms, symmetries and limits that the paper or elementary algebra fix.
"""
import math

import numpy as np
import pytest

from oracle import lapsum_oracle as O


def sigma(u):
    u = np.asarray(u, dtype=np.float64)
    return np.where(u <= 0, 0.5 * np.exp(np.minimum(u, 0)), 1 - 0.5 * np.exp(-np.maximum(u, 0)))


def lap_numpy(r, b, t):
    return float(np.sum(sigma((np.asarray(r, np.float64) - b) / t)))


def tiny_cases():
    rng = np.random.default_rng(7)
    cases = []
    for trial in range(120):
        n = int(rng.integers(1, 65))
        r = rng.standard_normal(n).astype(np.float32) * float(rng.choice([0.2, 1.0, 5.0]))
        if trial % 3 == 0 and n > 3:  # exact ties
            r[rng.integers(0, n, n // 2)] = r[rng.integers(0, n)]
        if trial % 4 == 0:
            k = float(rng.uniform(0.05, n - 0.05))  # non-integer budgets
        else:
            k = float(rng.integers(1, n)) if n > 1 else 0.5
        t = float(rng.choice([0.05, 0.3, 1.0, 3.0]))
        cases.append((r, k, -t))
    return cases


def test_lap_sum_is_the_plain_definition():
    rng = np.random.default_rng(0)
    r = rng.standard_normal(200).astype(np.float32)
    for b in (-1.0, 0.0, 0.37, 2.0):
        assert O.lap_sum(r, b, 0.4) == pytest.approx(lap_numpy(r, b, 0.4), rel=1e-13)
    # sigma(0) = 1/2, far above -> 1, far below -> 0 (Eq. 3)
    assert O.lap_sum(np.zeros(1, np.float32), 0.0, 1.0) == 0.5
    assert O.lap_sum(np.full(1, 50.0, np.float32), 0.0, 1.0) == pytest.approx(1.0, abs=1e-15)
    assert O.lap_sum(np.full(1, -50.0, np.float32), 0.0, 1.0) == pytest.approx(0.0, abs=1e-15)


def test_forward_matches_full_sum_bisection_on_tiny_inputs():
    worst_p, worst_res = 0.0, 0.0
    for r, k, alpha in tiny_cases():
        t = -alpha
        f = O.forward(r, k, alpha)
        b_bis = O.bisect(r, k, alpha)
        p_bis = sigma((r.astype(np.float64) - b_bis) / t)
        worst_p = max(worst_p, float(np.max(np.abs(f.p[0] - p_bis))))
        worst_res = max(worst_res, abs(lap_numpy(r, f.b[0], t) - k) / k)
    assert worst_p <= 1e-12
    assert worst_res <= 1e-12


def test_b_matches_bisection_when_well_conditioned():
    rng = np.random.default_rng(3)
    for _ in range(40):
        n = int(rng.integers(8, 64))
        r = rng.standard_normal(n).astype(np.float32)
        k = float(rng.uniform(0.5, n - 0.5))  # non-integer: no plateau
        f = O.forward(r, k, -0.5)
        assert f.b[0] == pytest.approx(O.bisect(r, k, -0.5), abs=1e-11)


def test_budget_and_range_and_monotonicity():
    for r, k, alpha in tiny_cases():
        f = O.forward(r, k, alpha)
        p = f.p[0]
        assert abs(p.sum() - k) <= 1e-11 * max(1.0, k)
        assert np.all(p >= 0) and np.all(p <= 1)
        near = np.abs(r.astype(np.float64) - f.b[0]) / (-alpha) < 30
        assert np.all(p[near] > 0) and np.all(p[near] < 1)
        order = np.argsort(r, kind="stable")
        assert np.all(np.diff(p[order]) >= 0)  # r_i <= r_j  =>  p_i <= p_j


def test_single_score_closed_form():
    # n = 1: sigma((r-b)/t) = k  =>  b = r - t ln(2k) (k <= 1/2),  b = r + t ln(2(1-k)) (k > 1/2)
    for r0, k, t in [(0.3, 0.2, 0.7), (-1.5, 0.5, 0.1), (2.0, 0.9, 1.3)]:
        r = np.array([r0], np.float32)
        b = O.forward(r, k, -t).b[0]
        want = float(r[0]) - t * math.log(2 * k) if k <= 0.5 else float(r[0]) + t * math.log(2 * (1 - k))
        assert b == pytest.approx(want, abs=1e-13)


def test_all_equal_scores_closed_form():
    # every p_i = k/n, so b = c - t * sigma^{-1}(k/n)
    for n, k, t, c in [(16, 3.0, 0.5, 0.75), (64, 40.0, 0.05, -2.0), (33, 16.5, 1.0, 0.0)]:
        r = np.full(n, c, np.float32)
        f = O.forward(r, k, -t)
        assert np.allclose(f.p[0], k / n, atol=1e-14)
        q = k / n
        inv = math.log(2 * q) if q <= 0.5 else -math.log(2 * (1 - q))
        assert f.b[0] == pytest.approx(float(np.float32(c)) - t * inv, abs=1e-12)


def test_symmetric_scores_half_budget():
    # scores symmetric about c with k = n/2: b = c exactly and p_i + p_mirror(i) = 1
    rng = np.random.default_rng(11)
    half = (rng.integers(1, 1500, 20) / 512.0).astype(np.float32)  # exact in fp32, so the mirror is exact
    c = np.float32(0.5)
    r = np.concatenate([c + np.abs(half), c - np.abs(half)]).astype(np.float32)
    n = r.shape[0]
    f = O.forward(r, n / 2, -0.3)
    assert f.b[0] == pytest.approx(float(c), abs=1e-12)
    assert np.allclose(f.p[0][:20] + f.p[0][20:], 1.0, atol=1e-12)


def test_zero_temperature_limit_is_the_midpoint():
    # Theorem 1: distinct scores, integer k, t -> 0: b -> (r_(k) + r_(k+1))/2, p -> hard top-k
    rng = np.random.default_rng(5)
    r = rng.permutation(np.arange(40)).astype(np.float32) * 0.37
    k = 7
    desc = np.sort(r.astype(np.float64))[::-1]
    mid = 0.5 * (desc[k - 1] + desc[k])
    errs = []
    for t in (0.05, 0.01, 0.002):
        f = O.forward(r, k, -t)
        errs.append(abs(f.b[0] - mid))
    assert errs[-1] <= 1e-9
    f = O.forward(r, k, -0.002)
    hard = (r > mid).astype(np.float64)
    assert np.max(np.abs(f.p[0] - hard)) < 1e-12
    assert hard.sum() == k


def test_shift_and_scale_invariance():
    rng = np.random.default_rng(2)
    # powers of two keep the fp32 inputs exactly related
    r = (rng.integers(-2000, 2000, 48) / 256.0).astype(np.float32)
    k, t = 9.0, 0.25
    f0 = O.forward(r, k, -t)
    f1 = O.forward(r + np.float32(4.0), k, -t)
    assert np.allclose(f0.p, f1.p, atol=1e-13)
    assert f1.b[0] == pytest.approx(f0.b[0] + 4.0, abs=1e-12)
    f2 = O.forward(r * np.float32(2.0), k, -2 * t)
    assert np.allclose(f0.p, f2.p, atol=1e-13)
    assert f2.b[0] == pytest.approx(2 * f0.b[0], abs=1e-12)


def test_node_values_equal_brute_force_sums():
    rng = np.random.default_rng(9)
    for n, t in [(1, 0.5), (2, 0.1), (17, 0.3), (40, 1.0)]:
        r = rng.standard_normal(n).astype(np.float32)
        if n > 10:
            r[3] = r[8]
        k = max(0.5, n / 3)
        f = O.forward(r, k, -t, want_nodes=True)
        s = np.sort(r.astype(np.float64))
        for m in range(1, n + 1):
            assert f.node_F[0, m] == pytest.approx(lap_numpy(r, s[m - 1], t), rel=1e-12, abs=1e-12)
        assert f.node_F[0, 0] == math.inf and f.node_F[0, n + 1] == -math.inf
        # j* = number of nodes whose value is >= k (F is non-increasing along the sorted nodes)
        assert f.jstar[0] == int(np.sum(f.node_F[0, 1 : n + 1] >= k))


def test_two_pivot_forms_of_the_root_agree():
    # the quadratic in u = e^{(b-lo)/t} and the one in w = e^{(hi-b)/t} have the same root:
    # shifting k by a hair flips the branch (c changes sign at integer crossings)
    rng = np.random.default_rng(13)
    for _ in range(30):
        x = np.sort(rng.standard_normal(30))
        t = 0.4
        s = O.solve_sorted(x, 12.0, t)
        u_form = s.lo + t * math.log(s.A / (math.sqrt(s.c ** 2 + s.A * s.Bs * math.exp(-(s.hi - s.lo) / t)) - s.c))
        w_form = s.hi - t * math.log(s.Bs / (s.c + math.sqrt(s.c ** 2 + s.A * math.exp(-(s.hi - s.lo) / t) * s.Bs)))
        assert u_form == pytest.approx(w_form, abs=1e-12)
        assert s.b == pytest.approx(u_form, abs=1e-12)
        assert s.lo <= s.b <= s.hi


def test_seeded_solve_equals_full_solve_for_any_bracket():
    # App. B: for any [a_L, a_R) that contains b the bracketed solve returns the same b
    rng = np.random.default_rng(17)
    for trial in range(60):
        n = int(rng.integers(5, 200))
        r = rng.standard_normal(n).astype(np.float32)
        if trial % 5 == 0:
            r[: n // 2] = r[0]
        k = float(rng.uniform(0.3, n - 0.3)) if trial % 2 else float(rng.integers(1, n))
        t = float(rng.choice([0.05, 0.5, 2.0]))
        full = O.forward(r, k, -t)
        b = full.b[0]
        wl, wr = rng.uniform(0.0, 2.0, 2)
        mode = trial % 4
        a_L = -np.inf if mode == 1 else np.float32(b - wl)
        a_R = np.inf if mode == 2 else np.float32(b + wr + 1e-3)
        if mode == 3:  # empty middle set
            srt = np.sort(r)
            i = np.searchsorted(srt, b)
            a_L = np.float32(np.nextafter(np.float32(srt[i - 1]), np.float32(np.inf))) if i > 0 else -np.inf
            a_R = np.float32(srt[i]) if i < n else np.inf
            if not (a_L <= b < a_R):
                continue
        br = O.forward_bracketed(r, k, -t, a_L, a_R)
        assert br.status == 0
        assert br.n_L + br.n_M + br.n_R == n
        if mode == 3:
            assert br.n_M == 0
        assert br.b == pytest.approx(b, abs=1e-11 * max(1.0, t))
        assert np.max(np.abs(br.p - full.p[0])) <= 1e-11


def test_failed_certificate_reports_the_side():
    rng = np.random.default_rng(19)
    r = rng.standard_normal(300).astype(np.float32)
    k, t = 20.0, 0.1
    b = O.forward(r, k, -t).b[0]
    left = O.forward_bracketed(r, k, -t, np.float32(b + 0.2), np.float32(b + 0.5))
    assert left.status == O.ROOT_LEFT  # Lap(a_L) < k
    right = O.forward_bracketed(r, k, -t, np.float32(b - 0.5), np.float32(b - 0.2))
    assert right.status == O.ROOT_RIGHT  # Lap(a_R) > k
    # the reported side matches the plain definition of Lap at the bracket ends
    assert lap_numpy(r, float(np.float32(b + 0.2)), t) < k
    assert lap_numpy(r, float(np.float32(b - 0.2)), t) > k


def test_sort_pairs_total_order_and_stability():
    r = np.array([0.0, -0.0, 1.5, -2.0, 1.5, np.float32(1e-45), -np.float32(1e-45), 3.0, -2.0], np.float32)
    keys, idx = O.sort_pairs(r)
    assert np.array_equal(keys.view(np.uint32), r[idx].view(np.uint32))
    assert list(idx) == [3, 8, 6, 1, 0, 5, 2, 4, 7]  # -0.0 before +0.0, ties by index
    rng = np.random.default_rng(23)
    x = rng.standard_normal(5000).astype(np.float32)
    x[rng.integers(0, 5000, 500)] = x[17]
    keys, idx = O.sort_pairs(x)
    ref = np.argsort(x, kind="stable")
    assert np.array_equal(idx, ref.astype(np.uint32))
    assert np.array_equal(keys, x[ref])


def test_budget_error_level_printed_by_the_paper():
    # Table "budget": |sum p - k|/k < 1e-5 (fp32) at k = N/16, alpha = -1, Gaussian; in fp64 far below
    rng = np.random.default_rng(29)
    for n in (1000, 10000, 100000):
        r = rng.standard_normal(n).astype(np.float32)
        f = O.forward(r, n / 16, -1.0)
        assert abs(f.p.sum() - n / 16) / (n / 16) < 1e-12
