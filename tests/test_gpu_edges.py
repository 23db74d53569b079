"""GPU edge cases: unaligned rows, several long rows, fractional budgets, extreme temperatures, the longest row."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import DeviceRun, assert_backward_matches, assert_forward_matches

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("path", [L.PATH_FULLSORT, L.PATH_BRACKET])
def test_rows_that_are_not_16_byte_aligned(path):
    # n odd: every second row starts off a 16-byte boundary, so the kernels take their scalar loads
    rows, n = 3, 70_001
    rng = np.random.default_rng(77)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    run = DeviceRun(r, 333.5, -0.07, L.default_params(force_path=path), seed=4).forward()
    assert run.status().status_bits == 0
    ref = assert_forward_matches(run, what=f"unaligned rows path={path}")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=f"unaligned rows path={path}")


@pytest.mark.parametrize("k", [0.25, 1.0, 17.3, 99_999.5])
def test_fractional_and_extreme_budgets_through_the_bracket(k):
    n = 100_000
    r = I.stress_row("gaussian", 9, n)
    run = DeviceRun(r, k, -0.05, L.default_params(force_path=L.PATH_BRACKET), seed=2).forward()
    assert_forward_matches(run, what=f"k={k}")


@pytest.mark.parametrize("alpha", [-1e-4, -1e-3, -10.0, -1e3])
def test_extreme_temperatures(alpha):
    for n, path in [(4096, L.PATH_AUTO), (200_000, L.PATH_FULLSORT), (200_000, L.PATH_BRACKET)]:
        r = I.stress_row("gaussian", 5, n)
        v = I.upstream(6, 1, n)
        run = DeviceRun(r, n / 50, alpha, L.default_params(force_path=path), seed=1).forward()
        ref = assert_forward_matches(run, what=f"alpha={alpha} n={n} path={path}")
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=f"alpha={alpha} n={n}")


def test_workspace_is_bound_to_its_shape_and_errors_are_synchronous():
    ws = L.Workspace(2, 1000)
    r = torch.zeros(3, 1000, device="cuda")
    p, b = torch.empty_like(r), torch.empty(3, device="cuda")
    with pytest.raises(L.LapsumError) as e:
        L.lapsum_forward(r, 10.0, -1.0, p, b, ws)
    assert e.value.code == -5
    r2 = torch.zeros(2, 1000, device="cuda")
    p2, b2 = torch.empty_like(r2), torch.empty(2, device="cuda")
    for k, alpha, code in [(0.0, -1.0, -3), (1000.0, -1.0, -3), (5.0, 0.0, -4), (5.0, float("inf"), -4)]:
        with pytest.raises(L.LapsumError) as e:
            L.lapsum_forward(r2, k, alpha, p2, b2, ws)
        assert e.value.code == code
    ws.release()
    with pytest.raises(L.LapsumError):
        L.lapsum_forward(r2, 5.0, -1.0, p2, b2, ws)


def test_profiling_hooks_count_every_launch():
    w = I.scaled(I.WORKLOADS["c4"], 300_000)
    run = DeviceRun(I.make_scores(w), w.k, w.alpha, None, seed=3)
    L.lapsum_profile_enable(run.ws, None, 256)
    before = L.lapsum_launch_count()
    run.forward().backward(I.make_upstream(w))
    launched = L.lapsum_launch_count() - before
    prof = L.lapsum_profile_read(run.ws)
    L.lapsum_profile_disable(run.ws)
    assert sum(nl for nl, _ in prof.values()) == launched
    assert {"stream_band", "cdf_map", "vjp_reduce", "vjp_map"} <= set(prof)
    assert all(ms > 0 for _, ms in prof.values())


def test_longest_row():
    # n = 2^30 - 1, the largest row the library accepts.  No oracle at this size: the threshold is checked against
    # the plain definition, sum_i sigma((r_i - b)/t) = k, evaluated with independent torch fp64 reductions.
    n = (1 << 30) - 1
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs about 30 GB of device memory")
    k, alpha = 250_000.0, -0.02
    t = -alpha
    g = torch.Generator(device="cuda").manual_seed(1234)
    r = torch.empty(1, n, device="cuda")
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        r[0, lo:hi].normal_(generator=g)
    p = torch.empty_like(r)
    b = torch.empty(1, device="cuda")
    ws = L.Workspace(1, n, None, seed=11)
    L.lapsum_forward(r, k, alpha, p, b, ws)
    torch.cuda.synchronize()
    st = ws.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0
    assert st.K == 1 << 20 and st.n_L + st.n_M + st.n_R == n
    bb = float(b[0])
    lap, total, lo_p, hi_p = 0.0, 0.0, 1.0, 0.0
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        u = (r[0, lo:hi].double() - bb) / t
        lap += float(torch.where(u <= 0, 0.5 * torch.exp(torch.clamp(u, max=0)), 1 - 0.5 * torch.exp(-torch.clamp(u, min=0))).sum())
        pc = p[0, lo:hi]
        total += float(pc.double().sum())
        lo_p, hi_p = min(lo_p, float(pc.min())), max(hi_p, float(pc.max()))
    assert abs(lap - k) <= 1e-4 * k          # b solves the budget equation
    assert abs(total - k) <= 1e-4 * k        # and the mask carries the budget
    assert 0.0 <= lo_p and hi_p <= 1.0
    # the mask is the CDF of the scores at that threshold (sampled positions)
    idx = torch.randint(0, n, (4096,), device="cuda", generator=g)
    u = (r[0, idx].double() - bb) / t
    want = torch.where(u <= 0, 0.5 * torch.exp(torch.clamp(u, max=0)), 1 - 0.5 * torch.exp(-torch.clamp(u, min=0)))
    assert float((p[0, idx].double() - want).abs().max()) <= 2e-6
    # backward at the same size: shift invariance and the closed form on sampled positions
    v = torch.empty_like(r)
    for lo in range(0, n, chunk):
        v[0, lo:min(n, lo + chunk)].normal_(generator=g)
    del p
    grad = torch.empty_like(r)
    L.lapsum_backward(v, r, b, k, alpha, grad, ws)
    torch.cuda.synchronize()
    s = ws.status()
    f = torch.exp(-(r[0, idx].double() - bb).abs() / t) / (2 * t)
    want_g = f * (v[0, idx].double() - s.S_vf / s.S_f)
    gmax = float(grad.abs().max())
    assert float((grad[0, idx].double() - want_g).abs().max()) <= 1e-4 * gmax
    assert abs(float(grad.double().sum())) <= 1e-3 * gmax


@pytest.mark.parametrize("kind", ["student_t2", "cauchy", "lognormal"])
@pytest.mark.parametrize("n,path", [(100, L.PATH_AUTO), (3000, L.PATH_AUTO), (50000, L.PATH_BRACKET), (50000, L.PATH_FULLSORT)])
def test_root_next_to_an_isolated_score_with_a_tiny_temperature(kind, n, path):
    # heavy tails, t far below the gaps between the top scores, fractional k: the root lies a fraction of t from one
    # score inside a gap of 1e5 t.  Its offset has to be kept against that score (the pivot of the form that applies);
    # measured from the far end of the gap it would be rounded at the gap's ulp, i.e. by a sizeable part of t
    rng = np.random.default_rng(n)
    rows = 3 if n <= 16384 else 1
    r = np.concatenate([I.stress_row(kind, 900 + i, n) for i in range(rows)], axis=0)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    for k in (4.614168, n - 4.614168, 1.5):
        run = DeviceRun(r, k, -1.7e-4, L.default_params(force_path=path), seed=4).forward()
        ref = assert_forward_matches(run, what=f"{kind} n={n} k={k}")
        run.backward(v)
        assert_backward_matches(run, v, ref.b, what=f"{kind} n={n} k={k}")


def test_two_host_threads_with_their_own_workspaces_and_streams():
    # the registry is behind one mutex and every call only enqueues: two threads, each with its own workspace and
    # stream, must not disturb each other (one long row on the bracket path, one batch on the block path)
    import threading

    jobs = [(I.stress_row("gaussian", 501, 300_000), 150.0, -0.05), (np.concatenate([I.stress_row("student_t2", 600 + i, 3000) for i in range(6)], 0), 40.0, -0.2)]
    refs = [O.forward(r, k, a) for r, k, a in jobs]
    errors = []

    def work(idx):
        try:
            r, k, a = jobs[idx]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                rd = torch.from_numpy(r).cuda()
                p, b = torch.empty_like(rd), torch.empty(r.shape[0], device="cuda")
            ws = L.Workspace(r.shape[0], r.shape[1], None, 3 + idx)
            for _ in range(25):
                L.lapsum_forward(rd, k, a, p, b, ws, stream)
            stream.synchronize()
            err = float(np.max(np.abs(p.cpu().numpy().astype(np.float64) - refs[idx].p)))
            if err > 2e-6:
                errors.append((idx, err))
        except Exception as e:  # noqa: BLE001
            errors.append((idx, repr(e)))

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
