"""The seeded generators: shapes, dtypes, determinism and the stated structure."""
import numpy as np

from paper_2608_06912_b200 import inputs as I


def test_workload_table():
    w = I.WORKLOADS
    assert (w["c1"].rows, w["c1"].n, w["c1"].k, w["c1"].alpha) == (4, 4096, 64.0, -0.05)
    assert (w["c2"].rows, w["c2"].n, w["c2"].k, w["c2"].alpha) == (65536, 128, 8.0, -0.1)
    assert (w["c3"].rows, w["c3"].n, w["c3"].k, w["c3"].alpha) == (1, 1 << 20, 210.0, -0.01)
    assert (w["c4"].rows, w["c4"].n, w["c4"].k, w["c4"].alpha) == (1, 10**7, 2000.0, -0.02)
    assert (w["c5"].rows, w["c5"].n, w["c5"].k, w["c5"].alpha) == (1, 10**8, 20000.0, -0.02)


def test_determinism_and_dtype():
    a = I.make_scores(I.WORKLOADS["c1"])
    b = I.make_scores(I.WORKLOADS["c1"])
    assert a.dtype == np.float32 and a.shape == (4, 4096) and a.flags.c_contiguous
    assert np.array_equal(a, b)
    v = I.make_upstream(I.WORKLOADS["c1"])
    assert v.shape == a.shape and not np.array_equal(a, v)


def test_duplicates_per_row():
    r = I.normal_rows_with_duplicates(5, 64, 128)
    for row in r:
        assert 128 - np.unique(row).shape[0] == 6  # round(0.05 * 128) duplicated values


def test_heavy_tail_mixture():
    r = I.heavy_tail_row(3, 1 << 18)[0]
    assert abs(np.mean(np.abs(r) > 0.5) - 0.1 * np.exp(-0.5)) < 0.01  # only the Laplace part reaches 0.5
    assert np.all(np.isfinite(r))


def test_scaled_keeps_budget_fraction():
    w = I.scaled(I.WORKLOADS["c5"], 10**6)
    assert w.n == 10**6 and w.k == 200.0 and w.alpha == -0.02
    r = I.make_scores(w)
    assert r.shape == (1, 10**6) and abs(float(r.std()) - 1.0) < 0.01


def test_stress_kinds():
    for kind in I.STRESS_KINDS + ("constant", "sorted_ramp"):
        r = I.stress_row(kind, 1, 4096)
        assert r.shape == (1, 4096) and r.dtype == np.float32 and np.all(np.isfinite(r))
    assert np.unique(I.stress_row("levels16", 1, 4096)).shape[0] == 16
