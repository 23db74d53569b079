"""Pins for the oracle's bracket: Eq. 8 indices, Theorem 2 coverage, Eq. 7 tails, sampler spec."""
import math
import os
from decimal import Decimal, getcontext

import numpy as np
import pytest
from scipy import stats

from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bracket_constants.txt")


def constants():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            key, val = line.split()
            out[key] = float(val)
    return out


def indices_by_decimal(n, k, z):
    """Eq. 8 with K = ceil(n^(2/3)), evaluated in 60-digit decimal arithmetic."""
    getcontext().prec = 60
    K = round(n ** (2.0 / 3.0))
    while K ** 3 < n * n:
        K += 1
    while (K - 1) ** 3 >= n * n:
        K -= 1
    q = (Decimal(n) - Decimal(k)) / Decimal(n)
    mu = Decimal(K) * q
    sd = (Decimal(K) * q * (1 - q)).sqrt()
    j = int((mu - Decimal(z) * sd).to_integral_value(rounding="ROUND_FLOOR"))
    l = int((mu + Decimal(z) * sd).to_integral_value(rounding="ROUND_CEILING"))
    return K, j, l


def test_printed_constants():
    c = constants()
    assert 2 * stats.norm.cdf(-c["z"]) == pytest.approx(c["miss_normal"], rel=0.05)
    assert 1 - 2 * stats.norm.cdf(-c["z99"]) >= c["coverage99"]
    assert O.sample_count(int(c["n_cube"])) == int(c["K_cube"])


@pytest.mark.parametrize("n,k", [(10**7, 2000), (10**8, 20000), (2**20, 210), (10**8, 10**8 // 16),
                                 (10**6, 62500), (12345, 17), (10**5, 99990)])
def test_indices_match_high_precision_evaluation(n, k):
    assert O.bracket_indices(n, k, 5.16) == indices_by_decimal(n, k, "5.16")


def test_known_index_values():
    # worked out by hand from Eq. 8 (z = 5.16)
    assert O.bracket_indices(10**7, 2000) == (46416, 46390, 46423)      # l > K: right end open
    assert O.bracket_indices(10**8, 20000) == (215444, 215367, 215435)
    assert O.bracket_indices(2**20, 210) == (10322, 10312, 10328)       # l > K
    assert O.bracket_indices(10**8, 10**8 / 16) == (215444, 201398, 202559)


def test_theorem2_coverage_with_iid_sampler():
    # Pr(y_(j) <= b < y_(l)) = Pr(j <= C <= l-1), C ~ Binomial(K, q): simulate the i.i.d. sampler
    rng = np.random.default_rng(5)
    n, k, t, z = 20000, 1500.0, 0.3, 1.0
    r = rng.standard_normal(n).astype(np.float32)
    b = O.forward(r, k, -t, want_p=False).b[0]
    K, j, l = O.bracket_indices(n, k, z)
    q = (n - k) / n
    want = stats.binom.cdf(l - 1, K, q) - stats.binom.cdf(j - 1, K, q)
    trials, hit = 3000, 0
    for _ in range(trials):
        y = np.sort(r[rng.integers(0, n, K)] + rng.laplace(0.0, t, K))
        hit += (y[j - 1] <= b < y[l - 1])
    se = math.sqrt(want * (1 - want) / trials)
    assert abs(hit / trials - want) < 4 * se + 1e-3


def test_systematic_sampler_spec():
    n = 100003
    K = O.sample_count(n)
    stride = n // K
    for seed in (0, 1, 0xDEADBEEF12345678):
        idx = O.sample_indices(seed, n, K)
        s = np.arange(K)
        assert np.all(idx >= s * stride) and np.all(idx < (s + 1) * stride)  # one draw per stratum
        e = O.noise_table(seed, K)
        assert e.dtype == np.float32 and np.all(np.isfinite(e))
    # unit Laplace: mean 0, E|e| = 1, median 0
    e = O.noise_table(12345, 200000).astype(np.float64)
    assert abs(e.mean()) < 0.02 and abs(np.abs(e).mean() - 1.0) < 0.02 and abs(np.median(e)) < 0.02
    # offsets inside the stride are spread out
    off = O.sample_indices(99, 10**7, O.sample_count(10**7)) % (10**7 // O.sample_count(10**7))
    assert abs(off.mean() / (10**7 // O.sample_count(10**7)) - 0.5) < 0.02


def test_bracket_sample_values_and_order_statistics():
    rng = np.random.default_rng(6)
    n, k, t, seed = 50000, 400.0, 0.05, 77
    r = rng.standard_normal(n).astype(np.float32)
    br = O.bracket(r, k, -t, 5.16, seed)
    K, j, l = O.bracket_indices(n, k, 5.16)
    assert (br.K, br.j, br.l) == (K, j, l)
    idx = O.sample_indices(seed, n, K)
    e = O.noise_table(seed, K)
    y64 = np.float32(t).astype(np.float64) * e.astype(np.float64) + r[idx].astype(np.float64)
    assert np.array_equal(br.y, y64.astype(np.float32))  # fma: one rounding of the exact value
    ys = np.sort(br.y)
    assert br.a_L == (ys[j - 1] if j >= 1 else -np.inf)
    assert br.a_R == (ys[l - 1] if l <= K else np.inf)
    # Eq. 7 and the partition, straight from the definition
    L = r < br.a_L
    R = r >= br.a_R
    assert (br.n_L, br.n_R, br.n_M) == (int(L.sum()), int(R.sum()), int(n - L.sum() - R.sum()))
    r64 = r.astype(np.float64)
    assert br.S_L == pytest.approx(np.exp((r64[L] - float(br.a_L)) / t).sum(), rel=1e-12)
    if R.any():
        assert br.S_R == pytest.approx(np.exp(-(r64[R] - float(br.a_R)) / t).sum(), rel=1e-12)
    else:
        assert br.S_R == 0.0


def test_systematic_sampler_coverage_over_seeds():
    # App. C, remark (iii): the systematic sampler's coverage is checked empirically
    rng = np.random.default_rng(8)
    n, k, t = 200000, 3000.0, 0.1
    r = rng.standard_normal(n).astype(np.float32)
    b = O.forward(r, k, -t, want_p=False).b[0]
    K, j, l = O.bracket_indices(n, k, 2.0)
    q = (n - k) / n
    want = stats.binom.cdf(l - 1, K, q) - stats.binom.cdf(j - 1, K, q)
    hits, trials = 0, 150
    for seed in range(trials):
        br = O.bracket(r, k, -t, 2.0, seed * 7919 + 1)
        hits += (br.a_L <= b < br.a_R)
    assert hits / trials > want - 0.08
    # at the operating point every seed brackets the root and the bracketed solve reproduces b
    for seed in range(5):
        br = O.bracket(r, k, -t, 5.16, seed)
        assert br.a_L <= b < br.a_R
        sol = O.forward_bracketed(r, k, -t, br.a_L, br.a_R, want_p=False)
        assert sol.status == 0 and sol.b == pytest.approx(b, abs=1e-11)
        assert (sol.n_L, sol.n_M, sol.n_R) == (br.n_L, br.n_M, br.n_R)


# ---- validated path: one-sided doubling before the full sort (App. C, expected-linear-time proposition) ----

def test_widen_moves_only_the_failing_side():
    # values exactly representable in fp32, so the expected ends are closed forms
    assert O.widen(1.0, 1.5, 0.125, 2) == (1.5, 2.5)       # root right: [a_R, a_R + 2 (a_R - a_L))
    assert O.widen(1.0, 1.5, 0.125, 1) == (0.0, 1.0)       # root left : [a_L - 2 (a_R - a_L), a_L)
    assert O.widen(1.0, 1.0, 0.25, 1) == (0.5, 1.0)        # empty bracket: the temperature stands in for the width
    assert O.widen(-np.inf, 2.0, 0.25, 2) == (2.0, 2.5)    # open on the far side: same
    assert O.widen(-np.inf, 2.0, 0.25, 1) is None          # nothing lies left of an open left end
    assert O.widen(2.0, np.inf, 0.25, 2) is None


@pytest.mark.parametrize("miss,width,expect", [
    (0.05, 0.15, 1),   # [b-0.2, b-0.05) -> [b-0.05, b+0.25)
    (0.40, 0.10, 2),   # [b-0.5, b-0.4) -> [b-0.4, b-0.2) -> [b-0.2, b+0.2)
    (0.95, 0.05, 3),   # widths 0.1, 0.2, 0.4 reach b-0.95+0.7 < b : needs a 4th -> with max 3 the full sort
])
@pytest.mark.parametrize("side", ["right", "left"])
def test_validated_path_counts_doublings_and_keeps_the_threshold(miss, width, expect, side):
    n, k, alpha = 20000, 150.0, -0.05
    r = I.stress_row("gaussian", 77, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    if side == "right":
        ends = (b - miss - width, b - miss)
    else:
        ends = (b + miss, b + miss + width)
    v = O.forward_validated(r, k, alpha, ends[0], ends[1], max_widen=3)
    # the doublings the geometry needs, stepped by hand (expect holds the count worked out on paper)
    lo, hi, m = np.float32(ends[0]), np.float32(ends[1]), 0
    while not (lo <= b < hi) and m < 3:
        w = hi - lo if hi > lo else np.float32(0.05)
        lo, hi = (hi, hi + 2 * w) if side == "right" else (lo - 2 * w, lo)
        m += 1
    assert v.widenings == m == expect
    assert v.full_sort == (not (lo <= b < hi))
    assert v.b == pytest.approx(b, abs=1e-12)
    assert np.allclose(v.p, ref.p[0], atol=1e-12)
    if not v.full_sort:
        rr = r[0]
        assert (v.n_L, v.n_M, v.n_R) == (int((rr < v.a_L).sum()), int(((rr >= v.a_L) & (rr < v.a_R)).sum()),
                                         int((rr >= v.a_R).sum()))


def test_validated_path_with_no_widenings_is_the_plain_fallback():
    n, k, alpha = 5000, 40.0, -0.1
    r = I.stress_row("gaussian", 78, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    v = O.forward_validated(r, k, alpha, b + 0.1, b + 0.2, max_widen=0)
    assert v.widenings == 0 and v.full_sort and v.b == pytest.approx(b, abs=1e-12)
