"""GPU parity of the gradients with respect to the budget k and the temperature alpha (all four backward kernels)."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import GRAD_RTOL, DeviceRun, to_dev

pytestmark = pytest.mark.gpu


def check(r, v, k, alpha, params=None, what=""):
    run = DeviceRun(r, k, alpha, params, seed=3).forward()
    rows = run.rows
    vv = to_dev(np.ascontiguousarray(v, np.float32).reshape(rows, run.n))
    g = torch.empty_like(run.r)
    gk = torch.full((rows,), float("nan"), device="cuda")
    ga = torch.full((rows,), float("nan"), device="cuda")
    L.lapsum_backward_scalars(vv, run.r, run.b, k, alpha, g, gk, ga, run.ws)
    torch.cuda.synchronize()
    ref = O.forward(run.r_np, k, alpha, want_p=False)
    gk_ref, ga_ref = O.backward_scalars(v, run.r_np, ref.b, alpha)
    g_ref = O.backward(v, run.r_np, ref.b, alpha)
    # grad_k is a weighted mean of v: scale = max|v|; grad_alpha: scale from the oracle's own magnitude
    vmax = np.abs(v).max()
    assert np.max(np.abs(gk.cpu().numpy() - gk_ref)) <= GRAD_RTOL * vmax, what
    scale_a = np.maximum(np.abs(ga_ref), 1e-3 * vmax * k / (-alpha))
    assert np.max(np.abs(ga.cpu().numpy() - ga_ref) / scale_a) <= 10 * GRAD_RTOL, what
    # the score gradient is unchanged by asking for the scalars
    g2 = torch.empty_like(run.r)
    L.lapsum_backward(vv, run.r, run.b, k, alpha, g2, run.ws)
    torch.cuda.synchronize()
    assert torch.equal(g, g2)
    assert np.max(np.abs(g.cpu().numpy() - g_ref)) <= GRAD_RTOL * np.max(np.abs(g_ref))
    # only one of the two may be requested
    gk2 = torch.empty(rows, device="cuda")
    L.lapsum_backward_scalars(vv, run.r, run.b, k, alpha, g2, gk2, None, run.ws)
    torch.cuda.synchronize()
    assert torch.equal(gk, gk2)


def test_warp_and_block_paths():
    rng = np.random.default_rng(1)
    for rows, n, k, alpha in [(257, 128, 8.0, -0.1), (33, 50, 5.5, -0.5), (4, 4096, 64.0, -0.05), (3, 1000, 62.5, -1.0)]:
        r = rng.standard_normal((rows, n)).astype(np.float32)
        v = rng.standard_normal((rows, n)).astype(np.float32)
        check(r, v, k, alpha, what=f"{rows}x{n}")


@pytest.mark.parametrize("path", [L.PATH_FULLSORT, L.PATH_BRACKET])
def test_long_rows(path):
    for name, n in [("c4", 300_000), ("c3", 1 << 18)]:
        w = I.scaled(I.WORKLOADS[name], n)
        check(I.make_scores(w), I.make_upstream(w), w.k, w.alpha, L.default_params(force_path=path), what=f"{name}@{n}")


def test_constant_upstream():
    # L = c * sum p = c k: dL/dk = c, dL/dalpha = 0
    w = I.scaled(I.WORKLOADS["c5"], 500_000)
    r = I.make_scores(w)
    run = DeviceRun(r, w.k, w.alpha, None, seed=1).forward()
    v = torch.full_like(run.r, 2.5)
    g, gk, ga = torch.empty_like(run.r), torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    L.lapsum_backward_scalars(v, run.r, run.b, w.k, w.alpha, g, gk, ga, run.ws)
    torch.cuda.synchronize()
    assert float(gk[0]) == pytest.approx(2.5, rel=1e-6)
    assert abs(float(ga[0])) <= 1e-3 * 2.5 * w.k / (-w.alpha) * 1e-3
