"""Seeded synthetic inputs for the LapSum soft top-k workloads.

This module only draws numbers.  It holds none of the method's arithmetic
(no CDF, no threshold, no sort keys), so both the CUDA path and the CPU oracle
may be fed from it without sharing any code of the method itself.

The five named workloads mirror the shapes, value distributions and budgets
the solver is specified on:

* ``c1`` rows=4, n=4096, N(0,1), k=64, alpha=-0.05
* ``c2`` rows=65536, n=128, N(0,1) with 5 % exact duplicates per row
  (MoE-routing shape), k=8, alpha=-0.1
* ``c3`` 1 x 1,048,576: each element Laplace(0, scale 1) with probability 0.1,
  otherwise N(0, std 0.1) (a saliency-map-like heavy tail), k=210, alpha=-0.01
* ``c4`` 1 x 10^7, N(0,1), k=2000, alpha=-0.02
* ``c5`` 1 x 10^8, N(0,1) + U(-1e-3, 1e-3) summed in fp64 then cast,
  k=20000, alpha=-0.02

All arrays are generated on the host with ``numpy.random.default_rng(seed)``
and returned as C-contiguous float32.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Callable, Dict

import numpy as np

_CHUNK = 1 << 24  # elements drawn per chunk for the very large rows


@dataclass(frozen=True)
class Workload:
    name: str
    rows: int
    n: int
    k: float
    alpha: float
    seed_r: int
    seed_v: int
    seed_sampler: int
    recipe: str

    @property
    def scores(self) -> int:
        return self.rows * self.n


def _normal_chunks(rng: np.random.Generator, n: int, post: Callable | None = None) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        x = rng.standard_normal(hi - lo)
        if post is not None:
            x = post(rng, x)
        out[lo:hi] = x.astype(np.float32)
    return out


def normal_rows(seed: int, rows: int, n: int) -> np.ndarray:
    """rows x n iid N(0,1) scores."""
    rng = np.random.default_rng(seed)
    return _normal_chunks(rng, rows * n).reshape(rows, n)


def normal_rows_with_duplicates(seed: int, rows: int, n: int, frac: float = 0.05) -> np.ndarray:
    """N(0,1) rows in which round(frac*n) positions of every row are
    overwritten with the value of another, untouched, position of the same
    row, so each row carries exact duplicates (ties)."""
    rng = np.random.default_rng(seed)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    d = int(round(frac * n))
    if d > 0 and 2 * d <= n:
        # a random permutation per row: first d positions are destinations,
        # the next d are the (untouched) sources
        perm = np.argsort(rng.random((rows, n)), axis=1)[:, : 2 * d]
        rr = np.arange(rows)[:, None]
        r[rr, perm[:, :d]] = r[rr, perm[:, d:]]
    return np.ascontiguousarray(r)


def heavy_tail_row(seed: int, n: int, p_tail: float = 0.1, std: float = 0.1) -> np.ndarray:
    """One row: Laplace(0, scale 1) with probability p_tail else N(0, std)."""
    rng = np.random.default_rng(seed)
    out = np.empty(n, dtype=np.float32)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        m = hi - lo
        is_tail = rng.random(m) < p_tail
        body = rng.standard_normal(m) * std
        tail = rng.laplace(0.0, 1.0, m)
        out[lo:hi] = np.where(is_tail, tail, body).astype(np.float32)
    return out.reshape(1, n)


def normal_plus_uniform_row(seed: int, n: int, half_width: float = 1e-3) -> np.ndarray:
    """One row: N(0,1) + U(-half_width, half_width), summed in fp64, cast to fp32."""
    rng = np.random.default_rng(seed)

    def post(g, x):
        return x + g.uniform(-half_width, half_width, x.shape[0])

    return _normal_chunks(rng, n, post).reshape(1, n)


def upstream(seed: int, rows: int, n: int) -> np.ndarray:
    """Upstream gradient v ~ N(0,1), same shape as the scores."""
    rng = np.random.default_rng(seed)
    return _normal_chunks(rng, rows * n).reshape(rows, n)


WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", 4, 4096, 64.0, -0.05, 1001, 2001, 3001, "N(0,1)"),
    "c2": Workload("c2", 65536, 128, 8.0, -0.1, 1002, 2002, 3002, "N(0,1), 5% exact duplicates per row"),
    "c3": Workload("c3", 1, 1 << 20, 210.0, -0.01, 1003, 2003, 3003, "0.9 N(0,std 0.1) + 0.1 Laplace(0,1)"),
    "c4": Workload("c4", 1, 10_000_000, 2000.0, -0.02, 1004, 2004, 3004, "N(0,1)"),
    "c5": Workload("c5", 1, 100_000_000, 20000.0, -0.02, 1005, 2005, 3005, "N(0,1)+U(-1e-3,1e-3)"),
}


# The paper's own benchmark grid (Table "Large-N summary": Gaussian scores, B = 1, k = N/16, alpha = -1)
for _n, _tag in ((10**6, "1e6"), (10**7, "1e7"), (10**8, "1e8")):
    WORKLOADS[f"paper{_tag}"] = Workload(f"paper{_tag}", 1, _n, _n / 16, -1.0, 1100 + len(_tag), 2100, 3100,
                                         "N(0,1), k=n/16, alpha=-1 (the paper's large-N grid)")


# The paper's small-batch grid (Table "forward time by problem size / batch / temperature / budget":
# Gaussian scores; one axis varies at a time around B = 8..16, n = 2048..4096, k = n/16, alpha = -1)
SMALL_BATCH_GRID = (
    [(8, n, n // 16, -1.0) for n in (256, 512, 1024, 2048, 4096, 8192, 16384)]
    + [(B, 4096, 256, -1.0) for B in (4, 16, 64, 256)]
    + [(16, 2048, 128, a) for a in (-0.25, -1.0, -4.0)]
    + [(16, 4096, k, -1.0) for k in (16, 256, 2048, 3840)]
)
for _B, _n, _k, _a in SMALL_BATCH_GRID:
    _name = f"grid_B{_B}_n{_n}_k{_k}_a{abs(_a):g}"
    WORKLOADS[_name] = Workload(_name, _B, _n, float(_k), _a, 1200 + _B + _n, 2200, 3200,
                                "N(0,1) (the paper's small-batch grid)")


# Batches of rows longer than the one-block-per-row path (not a shape of the paper's tables: its long rows come one at
# a time; per-sample budgets over images, Sec. 6, are the use): Gaussian rows, k = n/4096, alpha = -0.02
for _B, _n in ((8, 1 << 20), (64, 1 << 17), (4, 10_000_000)):
    _name = f"long_B{_B}_n{_n}"
    WORKLOADS[_name] = Workload(_name, _B, _n, float(_n // 4096), -0.02, 1300 + _B, 2300, 3300,
                                "N(0,1), a batch of long rows, k=n/4096")


def scaled(w: Workload, n: int) -> Workload:
    """The same recipe at another row length, with the budget kept at the same
    fraction k/n (used for reduced-size parity and profiling cases)."""
    k = max(1.0, float(round(w.k * n / w.n)))
    return replace(w, name=f"{w.name}@{n}", n=n, k=k)


def make_scores(w: Workload) -> np.ndarray:
    base = w.name.split("@")[0]
    if base == "c1":
        return normal_rows(w.seed_r, w.rows, w.n)
    if base == "c2":
        return normal_rows_with_duplicates(w.seed_r, w.rows, w.n)
    if base == "c3":
        return heavy_tail_row(w.seed_r, w.n)
    if base == "c4":
        return normal_rows(w.seed_r, w.rows, w.n)
    if base == "c5":
        return normal_plus_uniform_row(w.seed_r, w.n)
    if base.startswith("paper") or base.startswith("grid_") or base.startswith("long_"):
        return normal_rows(w.seed_r, w.rows, w.n)
    raise KeyError(w.name)


def make_upstream(w: Workload) -> np.ndarray:
    return upstream(w.seed_v, w.rows, w.n)


# ---- stress distributions (robustness table of the paper's Appendix C) ----

def stress_row(kind: str, seed: int, n: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    if kind == "gaussian":
        x = rng.standard_normal(n)
    elif kind == "student_t2":
        x = rng.standard_t(2.0, n)
    elif kind == "lognormal":
        x = rng.lognormal(0.0, 1.0, n)
    elif kind == "cauchy":
        x = np.clip(rng.standard_cauchy(n), -1e6, 1e6)
    elif kind == "clusters3":
        c = rng.integers(0, 3, n)
        x = np.array([-4.0, 0.0, 5.0])[c] + 0.3 * rng.standard_normal(n)
    elif kind == "levels16":
        x = rng.integers(0, 16, n).astype(np.float64) / 4.0
    elif kind == "constant":
        x = np.full(n, 0.75)
    elif kind == "sorted_ramp":
        x = np.linspace(-3.0, 3.0, n)
    else:
        raise KeyError(kind)
    return np.ascontiguousarray(x.astype(np.float32)).reshape(1, n)


STRESS_KINDS = ("gaussian", "student_t2", "lognormal", "cauchy", "clusters3", "levels16")
