"""GPU parity, full-sort path (global radix sort, tile scan, crossing-tile solve): C3, C4 and ragged sizes."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import DeviceRun, assert_backward_matches, assert_forward_matches, to_dev

pytestmark = pytest.mark.gpu

FULLSORT = dict(force_path=L.PATH_FULLSORT)


@pytest.mark.parametrize("n,k,alpha", [
    (16385, 100.0, -0.05), (20000, 1250.0, -1.0), (65536, 13.5, -0.02), (100003, 6250.0, -1.0),
    (262145, 52.0, -0.01), (8193 * 3 + 1, 12000.0, -0.3),
])
def test_ragged_sizes(n, k, alpha):
    rng = np.random.default_rng(n)
    r = rng.standard_normal((1, n)).astype(np.float32)
    v = rng.standard_normal((1, n)).astype(np.float32)
    run = DeviceRun(r, k, alpha, L.default_params(**FULLSORT)).forward()
    st = run.status()
    assert st.path == L.PATH_FULLSORT and st.status_bits == 0 and st.lookback_timeouts == 0
    ref = assert_forward_matches(run, what=f"n={n}")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=f"n={n}")


def test_several_rows_through_the_global_path():
    rng = np.random.default_rng(5)
    r = rng.standard_normal((3, 30000)).astype(np.float32)
    v = rng.standard_normal((3, 30000)).astype(np.float32)
    run = DeviceRun(r, 300.0, -0.1).forward()
    ref = assert_forward_matches(run, what="3x30000")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="3x30000")


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_config_full_sort(name):
    w = I.WORKLOADS[name]
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha, L.default_params(**FULLSORT)).forward()
    st = run.status()
    assert st.path == L.PATH_FULLSORT and st.status_bits == 0
    ref = assert_forward_matches(run, what=name)
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=name)
    # run-to-run determinism (fixed-order reductions)
    p0, b0, g0 = run.p.clone(), run.b.clone(), run.grad.clone()
    run.forward().backward(v)
    assert torch.equal(p0, run.p) and torch.equal(b0, run.b) and torch.equal(g0, run.grad)


@pytest.mark.parametrize("kind", I.STRESS_KINDS + ("constant", "sorted_ramp"))
def test_stress_distributions(kind):
    n = 200000
    r = I.stress_row(kind, 11, n)
    v = I.upstream(12, 1, n)
    for k, alpha in [(n / 16, -1.0), (50.0, -0.05)]:
        run = DeviceRun(r, k, alpha, L.default_params(**FULLSORT)).forward()
        ref = assert_forward_matches(run, what=f"{kind} k={k}")
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=kind)


@pytest.mark.parametrize("n", [16385, 100003, 1 << 20])
def test_radix_sort_pairs_bit_exact(n):
    rng = np.random.default_rng(n + 1)
    x = rng.standard_normal((1, n)).astype(np.float32)
    x[0, rng.integers(0, n, n // 4)] = x[0, 7]       # ties: stability shows in the payload
    x[0, 3], x[0, 4] = 0.0, -0.0
    ws = L.Workspace(1, n, L.default_params(sort_payload=1, **FULLSORT))
    keys_out = torch.empty((1, n), device="cuda", dtype=torch.float32)
    idx_out = torch.empty((1, n), device="cuda", dtype=torch.int32)
    L.lapsum_debug_sort_pairs(to_dev(x), keys_out, idx_out, ws)
    torch.cuda.synchronize()
    ko, io = O.sort_pairs(x[0])
    assert np.array_equal(keys_out.cpu().numpy()[0].view(np.uint32), ko.view(np.uint32))
    assert np.array_equal(idx_out.cpu().numpy()[0].view(np.uint32), io)
    assert ws.status().lookback_timeouts == 0


def test_payload_carrying_forward_equals_keys_only():
    n = 300000
    r = I.stress_row("gaussian", 3, n)
    a = DeviceRun(r, 1000.0, -0.05, L.default_params(**FULLSORT)).forward()
    b = DeviceRun(r, 1000.0, -0.05, L.default_params(sort_payload=1, **FULLSORT)).forward()
    assert torch.equal(a.p, b.p) and torch.equal(a.b, b.b)


@pytest.mark.parametrize("path", [L.PATH_AUTO, L.PATH_FULLSORT])
@pytest.mark.parametrize("rows,n", [(2, 20000), (5, 70001), (9, 300000), (37, 20011)])
def test_batches_of_long_rows_run_in_slots(rows, n, path):
    # rows > 1 on the long-row paths: up to sixteen rows at a time, each in its own copy of the per-call buffers (the
    # bracket path serves such a group with one launch per kernel, the full-sort path row by row on four streams);
    # thresholds, masks and gradients of every row against the oracle, twice on the same workspace, and the counters
    # summed over the slots.  37 rows: two full groups and a ragged one.
    rng = np.random.default_rng(rows * 1000 + n)
    r = np.concatenate([I.stress_row(kind, 70 + i, n) for i, kind in zip(range(rows), I.STRESS_KINDS * 7)], axis=0)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k, alpha = 0.003 * n, -0.05
    run = DeviceRun(r, k, alpha, L.default_params(force_path=path), seed=11)
    for _ in range(2):
        run.forward()
        ref = assert_forward_matches(run, what=f"{rows} rows of {n}")
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=f"{rows} rows of {n}")
    st = run.status()
    assert st.forwards == 2 and st.lookback_timeouts == 0 and not (st.status_bits & L.ST_LOOKBACK_TIMEOUT)
    assert st.path == (L.PATH_BRACKET if path == L.PATH_AUTO else L.PATH_FULLSORT)


@pytest.mark.parametrize("what", ["overflow", "narrow", "narrow_no_widening"])
def test_every_row_of_a_group_launches_its_own_repair(what):
    # one launch per kernel serves a group of rows; a row whose band overflows, or whose certificate fails, launches its
    # own full sort or its own widened attempt from the device, with its own slot's buffers.  Provoked from the host: a
    # band buffer of 64 scores (every row overflows), and z = 0.3 (most sampled brackets miss the root).
    rows, n = 21, 50_000
    rng = np.random.default_rng(77)
    r = rng.standard_normal((rows, n)).astype(np.float32) + np.arange(rows, dtype=np.float32)[:, None]
    v = rng.standard_normal((rows, n)).astype(np.float32)
    k, alpha = 300.0, -0.02
    prm = {"overflow": dict(band_capacity=64), "narrow": dict(z=0.3), "narrow_no_widening": dict(z=0.3, max_widenings=0)}[what]
    run = DeviceRun(r, k, alpha, L.default_params(force_path=L.PATH_BRACKET, **prm), seed=5)
    for _ in range(2):
        run.forward()
        ref = assert_forward_matches(run, what=what)
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=what)
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.forwards == 2 and st.lookback_timeouts == 0
    if what == "overflow":
        assert st.fallbacks == 2 * rows and st.status_bits & L.ST_BAND_OVERFLOW
    elif what == "narrow":
        assert st.widenings >= rows // 2          # z = 0.3 covers the root about one time in four
    else:
        assert st.widenings == 0 and st.fallbacks >= rows // 2


@pytest.mark.parametrize("path", [L.PATH_FULLSORT, L.PATH_BRACKET])
def test_a_lookback_wait_that_runs_out_reports_and_returns(path):
    # failure detection without a fault: one radix pass whose first tile is never processed (the ticket counter starts
    # at 1), so its counts are never published and every tile that needs them waits; the wait is bounded to a few hundred
    # polls here.  The kernel must return, raise the status bit and count the time-outs; the workspace must then serve
    # an exact forward + backward again without further time-outs.
    n, k, alpha = 100_003, 500.0, -0.05
    rng = np.random.default_rng(8)
    r = rng.standard_normal((1, n)).astype(np.float32)
    v = rng.standard_normal((1, n)).astype(np.float32)
    run = DeviceRun(r, k, alpha, L.default_params(force_path=path), seed=4).forward()
    assert run.status().lookback_timeouts == 0
    L.lapsum_debug_lookback_timeout(run.r, 300, run.ws)
    torch.cuda.synchronize()   # returns: nothing waits for ever
    st = run.status()
    assert st.status_bits & L.ST_LOOKBACK_TIMEOUT
    assert st.lookback_timeouts > 0
    timeouts = st.lookback_timeouts
    run.p.fill_(float("nan"))
    run.forward()
    ref = assert_forward_matches(run, what="forward after a time-out")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="backward after a time-out")
    assert run.status().lookback_timeouts == timeouts
    # a full-sort forward too (on the bracket workspace: through the sorted-keys hook, which runs the same chain)
    out = torch.empty_like(run.r)
    L.lapsum_debug_sort_pairs(run.r, out, None, run.ws)
    torch.cuda.synchronize()
    want, _ = O.sort_pairs(r[0])
    assert np.array_equal(out.cpu().numpy()[0].view(np.uint32), want.view(np.uint32))
    assert run.status().lookback_timeouts == timeouts
    with pytest.raises(L.LapsumError):
        L.lapsum_debug_lookback_timeout(run.r, 0, run.ws)          # the bound must be positive
