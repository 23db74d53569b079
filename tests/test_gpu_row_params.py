"""GPU parity of lapsum_forward_rows / lapsum_backward_rows: one budget and one temperature per row, on every path.

The paper's applications learn both k and alpha per sample (Sec. 6).  The oracle needs no new code: every row is its own
problem, solved by oracle.forward / oracle.backward / oracle.backward_scalars with the row's values."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from tests.gpu_util import B_RTOL, BUDGET_RTOL, GRAD_RTOL, P_ATOL, b_error

pytestmark = pytest.mark.gpu

SHAPES = [
    # rows, n, params, path expected
    (300, 100, {}, L.PATH_BLOCK),            # 16 lanes per row
    (40, 33, {}, L.PATH_BLOCK),
    (12, 1000, {}, L.PATH_BLOCK),            # one block per row
    (200, 700, {}, L.PATH_BLOCK),            # more rows than SMs
    (5, 4096, {}, L.PATH_BLOCK),             # cluster of four blocks per row
    (3, 16384, {}, L.PATH_BLOCK),            # cluster of eight
    (3, 70_001, {}, L.PATH_BRACKET),         # long rows: bracket path, radix selection
    (37, 20_011, {}, L.PATH_BRACKET),        # two full groups of 16 rows and a ragged one, one launch per kernel and group
    (2, 50_000, dict(full_sorts=1), L.PATH_BRACKET),
    (2, 30_000, dict(force_path=L.PATH_FULLSORT), L.PATH_FULLSORT),
    (1, 1 << 20, {}, L.PATH_BRACKET),
]


def draw(rng, rows, n):
    k = rng.uniform(0.3, n - 0.3, rows)
    whole = rng.random(rows) < 0.4
    k[whole] = np.clip(np.round(k[whole]), 1, max(1, n - 1))
    k[0] = max(1.0, n / 16)
    alpha = -(10.0 ** rng.uniform(-2.0, 0.3, rows))
    alpha[rng.random(rows) < 0.35] *= -1.0     # both signs in one batch
    alpha[0] = -0.05
    return k.astype(np.float64), alpha.astype(np.float64)


def run_rows(r, v, k, alpha, params, use_k=True, use_alpha=True, k_call=1.0, alpha_call=-1.0):
    rows, n = r.shape
    ws = L.Workspace(rows, n, L.default_params(**params), 5)
    rd, vd = torch.from_numpy(r).cuda(), torch.from_numpy(v).cuda()
    kd = torch.from_numpy(k).cuda() if use_k else None
    ad = torch.from_numpy(alpha).cuda() if use_alpha else None
    p, g = torch.full_like(rd, 7.0), torch.full_like(rd, 7.0)
    b = torch.full((rows,), 7.0, device="cuda")
    gk, ga = torch.full((rows,), 7.0, device="cuda"), torch.full((rows,), 7.0, device="cuda")
    L.lapsum_forward_rows(rd, kd, ad, k_call, alpha_call, p, b, ws)
    L.lapsum_backward_rows(vd, rd, b, ad, alpha_call, g, gk, ga, ws)
    torch.cuda.synchronize()
    return ws, p.cpu().numpy().astype(np.float64), b.cpu().numpy().astype(np.float64), \
        g.cpu().numpy().astype(np.float64), gk.cpu().numpy().astype(np.float64), ga.cpu().numpy().astype(np.float64)


def check_row(i, r, v, k, alpha, pg, bg, gg, gk, ga):
    ref = O.forward(r[i], k, alpha)
    assert np.max(np.abs(pg[i] - ref.p[0])) <= P_ATOL, (i, k, alpha)
    assert b_error(bg[i], ref.b, r[i], alpha) <= B_RTOL, (i, k, alpha)
    assert abs(pg[i].sum() - k) <= BUDGET_RTOL * k, (i, k, alpha)
    g_ref = O.backward(v[i], r[i], ref.b, alpha)[0]
    t = abs(alpha)
    f = np.exp(-np.abs(ref.b[0] - r[i].astype(np.float64)) / t) / (2 * t)
    scale = max(np.max(np.abs(g_ref)), 0.01 * f.max() * np.abs(v[i]).max(), 1e-30)
    assert np.max(np.abs(gg[i] - g_ref)) <= GRAD_RTOL * scale, (i, k, alpha)
    gk_ref, ga_ref = O.backward_scalars(v[i], r[i], ref.b, alpha)
    vmax = np.abs(v[i]).max()
    assert abs(gk[i] - gk_ref[0]) <= GRAD_RTOL * vmax, (i, k, alpha)
    scale_a = max(abs(ga_ref[0]), 1e-3 * vmax * min(k, len(r[i]) - k) / t)
    assert abs(ga[i] - ga_ref[0]) <= 10 * GRAD_RTOL * scale_a, (i, k, alpha, ga[i], ga_ref[0])


@pytest.mark.parametrize("rows,n,params,path", SHAPES)
def test_rows_with_their_own_budget_and_temperature(rows, n, params, path):
    rng = np.random.default_rng(rows * 131 + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k, alpha = draw(rng, rows, n)
    assert L.lapsum_describe(rows, n, params=L.default_params(**params)).path == path
    ws, pg, bg, gg, gk, ga = run_rows(r, v, k, alpha, params)
    st = ws.status()
    assert st.status_bits == 0 and st.path == path and st.fallbacks == 0
    for i in range(rows) if rows <= 40 else rng.choice(rows, 40, replace=False):
        check_row(i, r, v, k[i], alpha[i], pg, bg, gg, gk, ga)


@pytest.mark.parametrize("rows,n,params", [(33, 128, {}), (6, 3000, {}), (2, 40_000, {}), (2, 40_000, dict(force_path=L.PATH_FULLSORT))])
def test_one_vector_at_a_time_and_equal_rows_match_the_scalar_call(rows, n, params):
    rng = np.random.default_rng(n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k, alpha = draw(rng, rows, n)
    # budgets per row, shared temperature
    ws, pg, bg, gg, gk, ga = run_rows(r, v, k, alpha, params, use_alpha=False, alpha_call=0.3)
    for i in range(rows):
        check_row(i, r, v, k[i], 0.3, pg, bg, gg, gk, ga)
    # temperatures per row, shared budget
    ws, pg, bg, gg, gk, ga = run_rows(r, v, k, alpha, params, use_k=False, k_call=n / 8)
    for i in range(rows):
        check_row(i, r, v, n / 8, alpha[i], pg, bg, gg, gk, ga)
    # vectors of equal values: bit for bit what the scalar entry points give
    rd, vd = torch.from_numpy(r).cuda(), torch.from_numpy(v).cuda()
    ws = L.Workspace(rows, n, L.default_params(**params), 5)
    p1, g1, b1 = torch.empty_like(rd), torch.empty_like(rd), torch.empty(rows, device="cuda")
    p2, g2, b2 = torch.empty_like(rd), torch.empty_like(rd), torch.empty(rows, device="cuda")
    for a0 in (-0.2, 0.2):
        L.lapsum_forward(rd, n / 8, a0, p1, b1, ws)
        L.lapsum_backward(vd, rd, b1, n / 8, a0, g1, ws)
        kd = torch.full((rows,), n / 8, dtype=torch.float64, device="cuda")
        ad = torch.full((rows,), a0, dtype=torch.float64, device="cuda")
        L.lapsum_forward_rows(rd, kd, ad, 1.0, -1.0, p2, b2, ws)
        L.lapsum_backward_rows(vd, rd, b2, ad, -1.0, g2, None, None, ws)
        torch.cuda.synchronize()
        assert torch.equal(p1, p2) and torch.equal(b1, b2) and torch.equal(g1, g2)


@pytest.mark.parametrize("rows,n,params", [(8, 64, {}), (8, 1500, {}), (8, 4096, {}), (8, 20_000, {}),
                                           (8, 20_000, dict(full_sorts=1)), (8, 20_000, dict(force_path=L.PATH_FULLSORT))])
def test_a_bad_budget_or_temperature_voids_only_its_row(rows, n, params):
    rng = np.random.default_rng(rows + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k = np.full(rows, 5.0)
    alpha = np.full(rows, -0.1)
    k[1], k[3] = 0.0, float("nan")           # no root
    alpha[4], alpha[6] = 0.0, float("inf")   # no temperature
    k[6] = float(n)                          # both at once
    ws, pg, bg, gg, gk, ga = run_rows(r, v, k, alpha, params)
    st = ws.status()
    assert st.status_bits == (L.ST_BAD_BUDGET | L.ST_BAD_ALPHA), hex(st.status_bits)
    bad, good = [1, 3, 4, 6], [0, 2, 5, 7]
    assert np.isnan(bg[bad]).all() and np.isnan(pg[bad]).all()
    assert np.isnan(gg[[4, 6]]).all()        # the backward knows a bad temperature (the budget does not enter Eq. 5)
    for i in good:
        check_row(i, r, v, 5.0, -0.1, pg, bg, gg, gk, ga)
