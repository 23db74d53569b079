"""GPU parity for alpha > 0: Eq. 1 as printed, p_i = sigma((b - r_i)/alpha), the k smallest scores.  The CUDA path solves
the complementary problem (budget n - k) and complements the mask; the oracle solves on the negated scores: the two share
nothing but the definition.  Every path is covered: warp, block, cluster, full sort, bracket, host step, static backward."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import GRAD_RTOL, DeviceRun, assert_backward_matches, assert_forward_matches, to_dev

pytestmark = pytest.mark.gpu


def run_and_check(r, v, k, alpha, params=None, what=""):
    run = DeviceRun(r, k, alpha, params, seed=5).forward()
    ref = assert_forward_matches(run, what=what)
    run.backward(v)
    assert_backward_matches(run, np.asarray(v, np.float32).reshape(run.rows, run.n), ref.b, what=what)
    bits = run.status().status_bits
    assert bits & (L.ST_LOOKBACK_TIMEOUT | L.ST_NO_CROSSING) == 0, what
    return run, ref


@pytest.mark.parametrize("rows,n,k,alpha", [
    (300, 128, 8.0, 0.1),      # warp path, 4 items per lane
    (65, 31, 3.5, 0.5),        # warp path, 1 item per lane, ragged
    (7, 1000, 62.5, 1.0),      # one block per row
    (40, 2048, 128.0, 0.25),   # one block per row, many rows
    (4, 4096, 64.0, 0.05),     # cluster of four blocks per row
    (3, 16384, 1024.0, 1.0),   # cluster of eight blocks per row
    (2, 5000, 4999.0, 0.3),    # almost everything selected
    (2, 5000, 0.5, 0.3),       # less than one score selected
])
def test_short_rows(rows, n, k, alpha):
    rng = np.random.default_rng(rows * 1000 + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    run, ref = run_and_check(r, v, k, alpha, what=f"{rows}x{n} k={k} alpha={alpha}")
    # the mask falls as the score rises
    order = np.argsort(r[0], kind="stable")
    assert np.all(np.diff(run.p[0].cpu().numpy()[order]) <= 0)


@pytest.mark.parametrize("path", [L.PATH_FULLSORT, L.PATH_BRACKET])
@pytest.mark.parametrize("name,n", [("c4", 300_000), ("c3", 1 << 18), ("paper1e6", 1_000_000)])
def test_long_rows(path, name, n):
    w = I.scaled(I.WORKLOADS[name], n)
    r, v = I.make_scores(w), I.make_upstream(w)
    run, ref = run_and_check(r, v, w.k, -w.alpha, L.default_params(force_path=path), what=f"{name}@{n} path {path}")
    if path == L.PATH_BRACKET:
        # the bracket the device drew is that of the complementary problem: budget n - k at alpha' = -alpha
        st = run.status()
        if st.status_bits != 0:  # widened or fell back: the first bracket's counts are gone
            return
        br = O.bracket(r.reshape(-1), n - w.k, w.alpha, seed=5)
        assert (st.K, st.j, st.l) == (br.K, br.j, br.l)
        assert (st.n_L, st.n_M, st.n_R) == (br.n_L, br.n_M, br.n_R)


def test_mask_is_the_complement_of_the_negative_alpha_mask():
    rng = np.random.default_rng(8)
    for rows, n, k in [(5, 100, 7.0), (2, 3000, 200.5), (1, 400_000, 1234.0)]:
        r = rng.standard_normal((rows, n)).astype(np.float32)
        a = DeviceRun(r, k, 0.2, None, seed=2).forward()
        c = DeviceRun(r, n - k, -0.2, None, seed=2).forward()
        assert torch.equal(a.b, c.b)  # the same solve ran
        assert float((a.p - (1.0 - c.p)).abs().max()) <= 2e-7


def test_scalar_gradients():
    rng = np.random.default_rng(21)
    for rows, n, k, alpha, params in [(33, 50, 5.5, 0.5, None), (3, 1000, 62.5, 1.0, None), (4, 4096, 64.0, 0.05, None),
                                      (1, 300_000, 3000.0, 0.1, L.default_params(force_path=L.PATH_FULLSORT))]:
        r = rng.standard_normal((rows, n)).astype(np.float32)
        v = rng.standard_normal((rows, n)).astype(np.float32)
        run = DeviceRun(r, k, alpha, params, seed=3).forward()
        g = torch.empty_like(run.r)
        gk = torch.full((rows,), float("nan"), device="cuda")
        ga = torch.full((rows,), float("nan"), device="cuda")
        L.lapsum_backward_scalars(to_dev(v), run.r, run.b, k, alpha, g, gk, ga, run.ws)
        torch.cuda.synchronize()
        ref = O.forward(r, k, alpha, want_p=False)
        gk_ref, ga_ref = O.backward_scalars(v, r, ref.b, alpha)
        g_ref = O.backward(v, r, ref.b, alpha)
        vmax = np.abs(v).max()
        assert np.max(np.abs(gk.cpu().numpy() - gk_ref)) <= GRAD_RTOL * vmax
        scale_a = np.maximum(np.abs(ga_ref), 1e-3 * vmax * min(k, n - k) / alpha)
        assert np.max(np.abs(ga.cpu().numpy() - ga_ref) / scale_a) <= 10 * GRAD_RTOL
        assert np.max(np.abs(g.cpu().numpy() - g_ref)) <= GRAD_RTOL * np.max(np.abs(g_ref))


def test_host_step_and_static_backward():
    rng = np.random.default_rng(31)
    rows, n, k, alpha = 2, 200_000, 500.0, 0.05
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    run, ref = run_and_check(r, v, k, alpha, what="device step")
    r_h, v_h = torch.from_numpy(r).pin_memory(), torch.from_numpy(v).pin_memory()
    p_h, g_h, b_h = torch.zeros(rows, n).pin_memory(), torch.zeros(rows, n).pin_memory(), torch.zeros(rows).pin_memory()
    staging = torch.empty(4 * rows * n + rows, device="cuda")
    ws = L.Workspace(rows, n, None, 5)
    L.lapsum_forward_backward_host(r_h, v_h, k, alpha, p_h, g_h, b_h, staging, ws)
    torch.cuda.current_stream().synchronize()
    assert torch.equal(p_h, run.p.cpu()) and torch.equal(b_h, run.b.cpu()) and torch.equal(g_h, run.grad.cpu())
    g = torch.full_like(run.r, float("nan"))
    L.lapsum_backward_static(run.v, run.r, run.b, alpha, g)
    torch.cuda.synchronize()
    scale = float(run.grad.abs().max())
    assert float((g - run.grad).abs().max()) <= GRAD_RTOL * scale
