"""GPU parity, block path (one thread block per row, shared-memory bitonic sort): configs C1 and C2 and edge cases."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import DeviceRun, assert_backward_matches, assert_forward_matches, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_config_forward_backward(name):
    w = I.WORKLOADS[name]
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha).forward()
    st = run.status()
    assert st.path == L.PATH_BLOCK and st.status_bits == 0
    ref = assert_forward_matches(run, what=name)
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=name)


@pytest.mark.parametrize("rows,n,k,alpha", [
    (3, 1, 0.3, -0.5), (3, 2, 1.0, -0.2), (5, 3, 1.5, -1.0), (7, 5, 2.0, -0.05), (2, 31, 4.0, -0.1),
    (9, 100, 7.5, -0.3), (4, 129, 64.0, -0.02), (3, 1000, 62.5, -1.0), (2, 4097, 256.0, -0.05),
    (2, 8192, 512.0, -1.0), (2, 16384, 100.0, -0.01), (1, 16383, 16000.0, -0.5),
    # more rows than SMs: fewer threads per block, so 4, 8 and 8 keys per thread in the block sort
    (300, 200, 12.0, -0.1), (300, 700, 30.0, -0.05), (200, 3000, 100.0, -0.2), (150, 513, 500.0, -0.02),
])
def test_odd_shapes(rows, n, k, alpha):
    rng = np.random.default_rng(rows * 1000 + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    run = DeviceRun(r, k, alpha).forward()
    ref = assert_forward_matches(run, what=f"{rows}x{n}")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=f"{rows}x{n}")
    assert run.status().status_bits == 0


@pytest.mark.parametrize("B,n,k,alpha", I.SMALL_BATCH_GRID)
def test_papers_small_batch_grid(B, n, k, alpha):
    w = I.WORKLOADS[f"grid_B{B}_n{n}_k{k}_a{abs(alpha):g}"]
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha).forward()
    assert run.status().path == L.PATH_BLOCK
    ref = assert_forward_matches(run, what=w.name)
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=w.name)


@pytest.mark.parametrize("n", [1, 2, 7, 31, 32, 33, 63, 64, 65, 100, 127, 128])
def test_warp_path_row_lengths(n):
    # rows of up to 128 scores take the one-warp-per-row kernels; 1000 rows span several blocks and a ragged last one
    rng = np.random.default_rng(500 + n)
    rows = 1003
    r = rng.standard_normal((rows, n)).astype(np.float32)
    if n > 4:
        r[:, 1] = r[:, 3]  # a tie in every row
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k = 0.4 if n == 1 else max(1.0, n / 5)
    for alpha in (-0.1, -1.0):
        run = DeviceRun(r, k, alpha).forward()
        ref = assert_forward_matches(run, what=f"warp path n={n}")
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=f"warp path n={n}")
        assert run.status().status_bits == 0


def test_ties_and_degenerate_rows():
    n = 256
    rows = [
        np.full(n, 0.75, np.float32),                                        # all equal: p = k/n
        np.repeat(np.arange(16, dtype=np.float32) / 4, n // 16),             # 16 levels
        np.concatenate([np.zeros(n // 2, np.float32), -np.zeros(n // 2, np.float32)]),  # +0 / -0
        np.linspace(-3, 3, n).astype(np.float32),                            # already sorted
        np.linspace(3, -3, n).astype(np.float32),                            # reverse sorted
        np.concatenate([np.full(n - 1, -5.0, np.float32), [40.0]]).astype(np.float32),  # one outlier
    ]
    r = np.stack(rows)
    for k, alpha in [(8.0, -0.1), (100.5, -1.0), (255.0, -0.01)]:
        run = DeviceRun(r, k, alpha).forward()
        ref = O.forward(r, k, alpha)
        p = run.p.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(p - ref.p)) <= 2e-6
        assert np.max(np.abs(p.sum(axis=1) - k)) <= 1e-4 * k
        assert np.allclose(p[0], k / n, atol=2e-6)


def test_zero_temperature_plateau_gives_hard_topk():
    # gaps >> t: the mask is the hard top-k indicator (Theorem 1) whatever point of the plateau b is
    r = (np.random.default_rng(3).permutation(512).astype(np.float32) * 0.5).reshape(1, -1)
    run = DeviceRun(r, 20.0, -0.001).forward()
    p = run.p.cpu().numpy()[0]
    assert p.sum() == pytest.approx(20.0, abs=2e-3)
    assert np.array_equal(p > 0.5, r[0] >= np.sort(r[0])[-20])
    ref = O.forward(r, 20.0, -0.001)
    assert abs(float(run.b[0]) - ref.b[0]) <= 1e-5 * abs(ref.b[0])


@pytest.mark.parametrize("rows,n", [(1, 1), (5, 7), (16, 128), (3, 1000), (2, 4096), (2, 16384), (3, 5000)])
def test_sort_pairs_bit_exact(rows, n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal((rows, n)).astype(np.float32)
    if n > 8:
        x[:, rng.integers(0, n, n // 3)] = x[:, [0]]        # heavy ties
        x[:, 1] = 0.0
        x[:, 2] = -0.0
    ws = L.Workspace(rows, n)
    keys_out = torch.empty((rows, n), device="cuda", dtype=torch.float32)
    idx_out = torch.empty((rows, n), device="cuda", dtype=torch.int32)
    L.lapsum_debug_sort_pairs(to_dev(x), keys_out, idx_out, ws)
    torch.cuda.synchronize()
    kg = keys_out.cpu().numpy()
    ig = idx_out.cpu().numpy().view(np.uint32)
    for row in range(rows):
        ko, io = O.sort_pairs(x[row])
        assert np.array_equal(kg[row].view(np.uint32), ko.view(np.uint32))
        assert np.array_equal(ig[row], io)


def test_repeated_calls_are_bit_identical():
    w = I.WORKLOADS["c1"]
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha).forward().backward(v)
    p0, b0, g0 = run.p.clone(), run.b.clone(), run.grad.clone()
    for _ in range(3):
        run.forward().backward(v)
        assert torch.equal(p0, run.p) and torch.equal(b0, run.b) and torch.equal(g0, run.grad)


def test_mask_is_monotone_in_the_scores():
    w = I.WORKLOADS["c1"]
    r = I.make_scores(w)
    run = DeviceRun(r, w.k, w.alpha).forward()
    p = run.p.cpu().numpy()
    for row in range(w.rows):
        order = np.argsort(r[row], kind="stable")
        assert np.all(np.diff(p[row][order]) >= 0)


def test_shift_invariance_of_the_gradient():
    w = I.WORKLOADS["c1"]
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha).forward().backward(v)
    g = run.grad.double()
    assert float(g.sum(dim=1).abs().max()) <= 1e-4 * float(g.abs().max()) * 10
