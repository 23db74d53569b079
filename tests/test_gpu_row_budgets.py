"""GPU parity of lapsum_forward_row_budgets: one budget per row on the block path (warp, block and cluster kernels).
The oracle has no such entry point and needs none: each row is its own problem, solved by oracle.forward with its budget."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from tests.gpu_util import B_RTOL, BUDGET_RTOL, GRAD_RTOL, P_ATOL, b_error

pytestmark = pytest.mark.gpu


def draw_budgets(rng, rows, n):
    k = rng.uniform(0.3, n - 0.3, rows)
    whole = rng.random(rows) < 0.4
    k[whole] = np.clip(np.round(k[whole]), 1, max(1, n - 1))
    if n == 1:
        k = rng.uniform(0.1, 0.9, rows)
    return k.astype(np.float64)


@pytest.mark.parametrize("alpha", [-0.3, 0.3])
@pytest.mark.parametrize("rows,n", [(100, 7), (257, 128), (65, 50), (9, 1000), (40, 2048), (5, 4096), (3, 16384), (20, 8192)])
def test_rows_with_their_own_budgets(rows, n, alpha):
    rng = np.random.default_rng(rows * 31 + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k = draw_budgets(rng, rows, n)
    ws = L.Workspace(rows, n, None, 1)
    rd, vd, kd = torch.from_numpy(r).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(k).cuda()
    p, g, b = torch.empty_like(rd), torch.empty_like(rd), torch.empty(rows, device="cuda")
    gk = torch.empty(rows, device="cuda")
    L.lapsum_forward_row_budgets(rd, kd, alpha, p, b, ws)
    L.lapsum_backward_scalars(vd, rd, b, 1.0, alpha, g, gk, None, ws)
    torch.cuda.synchronize()
    assert ws.status().status_bits == 0
    pg, bg, gg = p.cpu().numpy().astype(np.float64), b.cpu().numpy().astype(np.float64), g.cpu().numpy().astype(np.float64)
    for i in range(rows):
        ref = O.forward(r[i], k[i], alpha)
        assert np.max(np.abs(pg[i] - ref.p[0])) <= P_ATOL, (i, k[i])
        assert b_error(bg[i], ref.b, r[i], alpha) <= B_RTOL, (i, k[i])
        assert abs(pg[i].sum() - k[i]) <= BUDGET_RTOL * k[i]
        g_ref = O.backward(v[i], r[i], ref.b, alpha)[0]
        assert np.max(np.abs(gg[i] - g_ref)) <= GRAD_RTOL * max(np.max(np.abs(g_ref)), 1e-30), (i, k[i])
        gk_ref, _ = O.backward_scalars(v[i], r[i], ref.b, alpha)
        assert abs(float(gk[i]) - gk_ref[0]) <= GRAD_RTOL * np.abs(v[i]).max()


def test_equal_budgets_give_what_the_shared_budget_gives():
    rng = np.random.default_rng(4)
    for rows, n, k in [(33, 100, 7.5), (6, 3000, 100.0), (2, 16000, 77.0)]:
        r = torch.from_numpy(rng.standard_normal((rows, n)).astype(np.float32)).cuda()
        ws = L.Workspace(rows, n, None, 1)
        p1, b1 = torch.empty_like(r), torch.empty(rows, device="cuda")
        p2, b2 = torch.empty_like(r), torch.empty(rows, device="cuda")
        for alpha in (-0.2, 0.2):
            L.lapsum_forward(r, k, alpha, p1, b1, ws)
            L.lapsum_forward_row_budgets(r, torch.full((rows,), k, dtype=torch.float64, device="cuda"), alpha, p2, b2, ws)
            torch.cuda.synchronize()
            assert torch.equal(p1, p2) and torch.equal(b1, b2)


def test_a_budget_outside_the_open_interval_voids_only_its_row():
    rng = np.random.default_rng(6)
    for rows, n in [(8, 64), (8, 1500), (8, 4096)]:
        r = rng.standard_normal((rows, n)).astype(np.float32)
        k = np.full(rows, 5.0)
        k[1], k[3], k[4], k[6] = 0.0, float(n), float("nan"), -2.0
        ws = L.Workspace(rows, n, None, 1)
        rd = torch.from_numpy(r).cuda()
        p, b = torch.empty_like(rd), torch.empty(rows, device="cuda")
        L.lapsum_forward_row_budgets(rd, torch.from_numpy(k).cuda(), -0.1, p, b, ws)
        torch.cuda.synchronize()
        assert ws.status().status_bits == L.ST_BAD_BUDGET
        bad, good = [1, 3, 4, 6], [0, 2, 5, 7]
        assert torch.isnan(b[bad]).all() and torch.isnan(p[bad]).all()
        ref = O.forward(r[good], 5.0, -0.1)
        assert np.max(np.abs(p[good].cpu().numpy() - ref.p)) <= P_ATOL
        assert torch.isfinite(b[good]).all()


def test_long_rows_take_their_own_budgets_too():
    # rows beyond the block path: Eq. 8's ranks are formed on the device from each row's budget
    rng = np.random.default_rng(8)
    rows, n = 3, 100_000
    r = rng.standard_normal((rows, n)).astype(np.float32)
    k = np.array([5.0, 40_000.5, 99_000.0])
    ws = L.Workspace(rows, n, None, 1)
    rd = torch.from_numpy(r).cuda()
    p, b = torch.empty_like(rd), torch.empty(rows, device="cuda")
    L.lapsum_forward_row_budgets(rd, torch.from_numpy(k).cuda(), -0.1, p, b, ws)
    torch.cuda.synchronize()
    assert ws.status().status_bits == 0 and ws.status().path == L.PATH_BRACKET
    for i in range(rows):
        ref = O.forward(r[i], k[i], -0.1)
        assert np.max(np.abs(p[i].cpu().numpy() - ref.p[0])) <= P_ATOL
        assert b_error(float(b[i]), ref.b, r[i], -0.1) <= B_RTOL
