"""GPU parity, bracket path (sample, order statistics, stream pass, band sort, seeded solve, fallback)."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from paper_2608_06912_b200.binding import band_capacity
from tests.gpu_util import B_RTOL, DeviceRun, assert_backward_matches, assert_forward_matches, b_error, to_dev

pytestmark = pytest.mark.gpu

BRACKET = dict(force_path=L.PATH_BRACKET)


def check_bracket_stage(r, k, alpha, seed, z=5.16, full_sorts=0):
    """sample values, bracket ends and band counts bit-exact; tail sums to fp32 accuracy"""
    n = r.shape[1]
    ws = L.Workspace(1, n, L.default_params(z=z, full_sorts=full_sorts, **BRACKET), seed)
    K = O.sample_count(n)
    y = torch.empty(K, device="cuda")
    band = torch.full((band_capacity(ws),), float("nan"), device="cuda")
    L.lapsum_debug_bracket(to_dev(r), k, alpha, ws, y_out=y, band_out=band)
    st = ws.status()
    ref = O.bracket(r, k, alpha, z, seed)
    assert (st.K, st.j, st.l) == (ref.K, ref.j, ref.l)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), ref.y.view(np.uint32))
    assert np.float32(st.a_L).view(np.uint32) == np.float32(ref.a_L).view(np.uint32)
    assert np.float32(st.a_R).view(np.uint32) == np.float32(ref.a_R).view(np.uint32)
    assert (st.n_L, st.n_M, st.n_R) == (ref.n_L, ref.n_M, ref.n_R)
    assert st.S_L == pytest.approx(ref.S_L, rel=2e-6)
    assert st.S_R == pytest.approx(ref.S_R, rel=2e-6, abs=1e-30)
    if ref.n_M <= band.numel():  # otherwise the band overflowed its buffer (the forward then falls back)
        got = np.sort(band.cpu().numpy()[: ref.n_M])
        rr = r[0]
        want = np.sort(rr[(rr >= ref.a_L) & (rr < ref.a_R)])
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    return ref


@pytest.mark.parametrize("full_sorts", [0, 1])
@pytest.mark.parametrize("n,k,alpha,seed", [(4096, 256.0, -1.0, 5), (16385, 9.5, -0.02, 6), (40000, 2500.0, -0.3, 7),
                                             (65536, 100.0, -0.05, 1), (100003, 6250.0, -1.0, 2),
                                             (1 << 20, 210.0, -0.01, 3), (3_000_001, 600.0, -0.02, 4)])
def test_bracket_stage_bit_exact(n, k, alpha, seed, full_sorts):
    r = I.stress_row("gaussian", seed, n)
    check_bracket_stage(r, k, alpha, seed, full_sorts=full_sorts)


@pytest.mark.parametrize("kind,alpha", [("constant", -1e-3), ("constant", -1e-6), ("levels16", -1e-4),
                                        ("levels16", -0.5), ("cauchy", -0.01)])
def test_order_statistics_by_selection_on_clustered_samples(kind, alpha):
    # thousands of sample keys share their leading bits: the radix selection has to refine more than once
    n = 1 << 20
    r = I.stress_row(kind, 7, n)
    for k in (n / 2, 300.0):
        check_bracket_stage(r, k, alpha, 13)


@pytest.mark.parametrize("full_sorts", [0, 1])
@pytest.mark.parametrize("n,k,alpha", [(4096, 256.0, -1.0), (16385, 9.5, -0.02), (20000, 19990.0, -0.05), (40000, 2500.0, -0.3),
                                       (65536, 100.0, -0.05), (100003, 6250.0, -1.0), (1 << 20, 210.0, -0.01),
                                        (3_000_001, 187500.0, -1.0), (2_000_000, 1_000_000.0, -0.3)])
def test_bracket_forward_backward(n, k, alpha, full_sorts):
    rng = np.random.default_rng(n)
    r = rng.standard_normal((1, n)).astype(np.float32)
    v = rng.standard_normal((1, n)).astype(np.float32)
    run = DeviceRun(r, k, alpha, L.default_params(full_sorts=full_sorts, **BRACKET), seed=9).forward()
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.status_bits == 0 and st.fallbacks == 0
    ref = assert_forward_matches(run, what=f"bracket n={n}")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=f"bracket n={n}")


def test_c4_full_sort_and_bracket_cross_check():
    w = I.WORKLOADS["c4"]
    r, v = I.make_scores(w), I.make_upstream(w)
    ref_b = check_bracket_stage(r, w.k, w.alpha, w.seed_sampler)
    assert (ref_b.K, ref_b.j, ref_b.l) == (46416, 46390, 46423) and ref_b.a_R == np.inf and ref_b.n_R == 0
    br = DeviceRun(r, w.k, w.alpha, L.default_params(**BRACKET), seed=w.seed_sampler).forward()
    st = br.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0
    ref = assert_forward_matches(br, what="c4 bracket")
    fs = DeviceRun(r, w.k, w.alpha, L.default_params(force_path=L.PATH_FULLSORT)).forward()
    # the two pipelines agree with each other far inside the oracle tolerance
    assert abs(float(br.b[0]) - float(fs.b[0])) <= 1e-6 * abs(float(fs.b[0]))
    assert float((br.p - fs.p).abs().max()) <= 2e-6
    br.backward(v)
    assert_backward_matches(br, v, ref.b, what="c4 bracket")
    # default dispatch takes the bracket at this size
    auto = DeviceRun(r, w.k, w.alpha, None, seed=w.seed_sampler).forward()
    assert auto.status().path == L.PATH_BRACKET and torch.equal(auto.p, br.p)


def test_c3_default_dispatch_takes_the_bracket():
    # on B200 the bracket path wins on every row longer than the block path, so the megapixel-map shape goes through it by default
    w = I.WORKLOADS["c3"]
    r, v = I.make_scores(w), I.make_upstream(w)
    check_bracket_stage(r, w.k, w.alpha, w.seed_sampler)
    run = DeviceRun(r, w.k, w.alpha, None, seed=w.seed_sampler).forward()
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0
    ref = assert_forward_matches(run, what="c3 bracket")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="c3 bracket")
    fs = DeviceRun(r, w.k, w.alpha, L.default_params(force_path=L.PATH_FULLSORT)).forward()
    assert abs(float(run.b[0]) - float(fs.b[0])) <= 1e-6 * abs(float(fs.b[0]))
    assert float((run.p - fs.p).abs().max()) <= 2e-6


@pytest.mark.parametrize("name", ["paper1e6", "paper1e7"])
def test_papers_own_grid(name):
    # k = n/16, alpha = -1: a wide kernel (every score matters to the tails) and a band of 10^4..10^5 scores
    w = I.WORKLOADS[name]
    r, v = I.make_scores(w), I.make_upstream(w)
    check_bracket_stage(r, w.k, w.alpha, w.seed_sampler)
    run = DeviceRun(r, w.k, w.alpha, None, seed=w.seed_sampler).forward()
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0
    ref = assert_forward_matches(run, what=name)
    # the paper's own accuracy claim for this grid: |sum p - k| / k < 1e-5 in fp32 (Table "budget")
    assert abs(float(run.p.double().sum()) - w.k) / w.k < 1e-5
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what=name)


def test_c5_bracket():
    w = I.WORKLOADS["c5"]
    r = I.make_scores(w)
    ref_b = check_bracket_stage(r, w.k, w.alpha, w.seed_sampler)
    assert (ref_b.K, ref_b.j, ref_b.l) == (215444, 215367, 215435)
    run = DeviceRun(r, w.k, w.alpha, None, seed=w.seed_sampler).forward()
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0
    ref = assert_forward_matches(run, what="c5")
    del ref.p
    v = I.make_upstream(w)
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="c5")
    # fallback count over 20 sampler seeds (expected 0), same threshold every time
    fallbacks = 0
    for seed in range(20):
        ws = L.Workspace(1, w.n, None, seed)
        b = torch.empty(1, device="cuda")
        L.lapsum_forward(run.r, w.k, w.alpha, run.p, b, ws)
        s = ws.status()
        fallbacks += s.fallbacks
        assert abs(float(b[0]) - ref.b[0]) <= 1e-5 * abs(ref.b[0])
        ws.release()
    assert fallbacks == 0


def test_papers_1e8_grid_point():
    # k = n/16, alpha = -1 at n = 10^8: a band of ~10^5 scores, solved by several blocks (the bench row "paper1e8")
    w = I.WORKLOADS["paper1e8"]
    r = I.make_scores(w)
    check_bracket_stage(r, w.k, w.alpha, w.seed_sampler)
    run = DeviceRun(r, w.k, w.alpha, None, seed=w.seed_sampler).forward()
    st = run.status()
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0 and st.status_bits == 0 and st.n_M >= 65536
    ref = assert_forward_matches(run, what="paper1e8")
    assert abs(float(run.p.double().sum()) - w.k) / w.k < 1e-5
    del ref.p
    v = I.make_upstream(w)
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="paper1e8")


@pytest.mark.parametrize("mode", ["fallback", "overflow", "widen"])
def test_device_launched_chains_finish_before_the_mask_every_time(mode):
    # The band solve launches the widened attempt and the full-sort chain from the device (tail launches); the mask
    # kernel behind it must see their threshold.  Several hundred host-provoked failures in a row, every mask and
    # threshold against the oracle, the outputs poisoned before each call.  Nothing here faults or hangs a GPU.
    n, k, alpha = 200_000, 300.0, -0.05
    r = I.stress_row("gaussian", 23, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    p_ref = torch.from_numpy(ref.p).cuda()
    if mode == "fallback":
        prm, brackets = L.default_params(max_widenings=0, **BRACKET), [(b + 0.05, b + 0.2), (b - 0.2, b - 0.05)]
    elif mode == "overflow":
        prm, brackets = L.default_params(band_capacity=64, **BRACKET), [(b - 0.5, b + 0.5)]
    else:
        prm, brackets = L.default_params(max_widenings=2, **BRACKET), [(b + 0.02, b + 0.05), (b - 0.05, b - 0.02)]
    run = DeviceRun(r, k, alpha, prm)
    calls = 300
    for i in range(calls):
        run.p.fill_(float("nan"))
        run.b.fill_(float("nan"))
        a_L, a_R = brackets[i % len(brackets)]
        L.lapsum_forward_with_bracket(run.r, k, alpha, a_L, a_R, run.p, run.b, run.ws)
        err = float((run.p.double() - p_ref).abs().max())   # nan if any score kept its poison
        assert err <= 2e-6, f"call {i}: max|dp| = {err}"
        assert b_error(float(run.b[0]), ref.b, r, alpha) <= B_RTOL, f"call {i}"
    st = run.status()
    if mode == "widen":
        assert st.widenings == calls and st.fallbacks == 0
    else:
        assert st.fallbacks == calls


@pytest.mark.parametrize("which", ["left", "right", "empty", "overflow"])
def test_forced_fallback_still_exact(which):
    # host-side injection: a bracket that misses the root (or a band that cannot hold M) must end in the full sort
    n, k, alpha = 500000, 400.0, -0.05
    r = I.stress_row("gaussian", 21, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    prm = L.default_params(max_widenings=0, **BRACKET)
    if which == "left":
        ends, bit = (b + 0.05, b + 0.2), L.ST_ROOT_LEFT
    elif which == "right":
        ends, bit = (b - 0.2, b - 0.05), L.ST_ROOT_RIGHT
    elif which == "empty":
        ends, bit = (b + 0.1, b + 0.1), L.ST_ROOT_LEFT
    else:
        prm = L.default_params(band_capacity=64, **BRACKET)
        ends, bit = (b - 0.5, b + 0.5), L.ST_BAND_OVERFLOW
    run = DeviceRun(r, k, alpha, prm)
    L.lapsum_forward_with_bracket(run.r, k, alpha, ends[0], ends[1], run.p, run.b, run.ws)
    torch.cuda.synchronize()
    st = run.status()
    assert st.fallbacks == 1 and (st.status_bits & L.ST_FALLBACK) and (st.status_bits & bit)
    assert st.widenings == 0 and not (st.status_bits & L.ST_WIDENED)
    assert_forward_matches(run, ref, what=f"fallback {which}")
    # a good bracket on the same workspace afterwards takes the fast path again
    L.lapsum_forward_with_bracket(run.r, k, alpha, b - 0.01, b + 0.01, run.p, run.b, run.ws)
    torch.cuda.synchronize()
    assert run.status().fallbacks == 1
    assert_forward_matches(run, ref, what="good bracket after fallback")


@pytest.mark.parametrize("max_widenings", [1, 2, 3])
@pytest.mark.parametrize("side", ["left", "right"])
@pytest.mark.parametrize("miss,width", [(0.05, 0.15), (0.40, 0.10), (0.95, 0.05), (0.07, 0.0)])
def test_validated_widening_before_the_full_sort(miss, width, side, max_widenings):
    # host-side injection of a bracket that misses: one-sided doubling (App. C) until the certificate holds,
    # the full sort once max_widenings is used up; same attempts, same last bracket and counts as the oracle
    n, k, alpha = 500000, 400.0, -0.05
    r = I.stress_row("gaussian", 21, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    ends = (b - miss - width, b - miss) if side == "right" else (b + miss, b + miss + width)
    want = O.forward_validated(r, k, alpha, ends[0], ends[1], max_widen=max_widenings, want_p=False)
    run = DeviceRun(r, k, alpha, L.default_params(max_widenings=max_widenings, **BRACKET))
    for _ in range(2):  # the second call starts from clean per-call state again
        before = run.status()
        L.lapsum_forward_with_bracket(run.r, k, alpha, ends[0], ends[1], run.p, run.b, run.ws)
        torch.cuda.synchronize()
        st = run.status()
        assert st.widenings - before.widenings == want.widenings
        assert st.fallbacks - before.fallbacks == int(want.full_sort)
        assert bool(st.status_bits & L.ST_WIDENED) == (want.widenings > 0)
        assert bool(st.status_bits & L.ST_FALLBACK) == want.full_sort
        assert np.float32(st.a_L) == np.float32(want.a_L) and np.float32(st.a_R) == np.float32(want.a_R)
        assert (st.n_L, st.n_M, st.n_R) == (want.n_L, want.n_M, want.n_R)
        assert_forward_matches(run, ref, what=f"widening {side} miss={miss}")


def test_widening_on_a_large_row_and_backward_after_it():
    w = I.scaled(I.WORKLOADS["c4"], 3_000_000)
    r, v = I.make_scores(w), I.make_upstream(w)
    ref = O.forward(r, w.k, w.alpha)
    b = float(ref.b[0])
    run = DeviceRun(r, w.k, w.alpha, L.default_params(**BRACKET))
    L.lapsum_forward_with_bracket(run.r, w.k, w.alpha, b - 0.03, b - 0.01, run.p, run.b, run.ws)
    torch.cuda.synchronize()
    st = run.status()
    assert st.widenings == 1 and st.fallbacks == 0
    assert_forward_matches(run, ref, what="widened c4")
    run.backward(v)
    assert_backward_matches(run, v, ref.b, what="backward after a widened forward")


def test_sampled_brackets_that_miss_are_widened_by_the_multi_block_solve():
    # a narrow bracket (z = 1.5 misses about one time in eight) on a row whose expected band is long enough for the
    # band solve to run with several blocks: misses must end in a widened attempt (relaunched from the device with
    # the same block count), never in a wrong threshold
    n, k, alpha = 16_000_000, 8_000_000.0, -0.3
    r = I.stress_row("gaussian", 61, n)
    ref = O.forward(r, k, alpha)
    widened = 0
    for seed in range(16):
        run = DeviceRun(r, k, alpha, L.default_params(z=1.5, **BRACKET), seed=seed).forward()
        st = run.status()
        assert st.fallbacks == 0
        widened += st.widenings
        b = float(run.b[0])
        assert b_error(b, ref.b, r, alpha) <= B_RTOL, (seed, b, ref.b[0])
        if st.widenings or seed == 0:
            assert_forward_matches(run, ref, what=f"z=1.5 seed {seed}")
    assert widened >= 1


def test_one_sided_and_tight_brackets():
    n, k, alpha = 400000, 1000.0, -0.02
    r = I.stress_row("gaussian", 31, n)
    ref = O.forward(r, k, alpha)
    b = float(ref.b[0])
    for ends in [(-np.inf, b + 0.05), (b - 0.05, np.inf), (b - 1e-4, b + 1e-4), (-np.inf, np.inf)]:
        prm = L.default_params(band_capacity=n, **BRACKET)
        run = DeviceRun(r, k, alpha, prm)
        L.lapsum_forward_with_bracket(run.r, k, alpha, ends[0], ends[1], run.p, run.b, run.ws)
        torch.cuda.synchronize()
        assert run.status().fallbacks == 0
        assert_forward_matches(run, ref, what=f"bracket {ends}")


@pytest.mark.parametrize("full_sorts", [0, 1])
@pytest.mark.parametrize("kind", I.STRESS_KINDS + ("constant",))
def test_stress_distributions_through_the_bracket(kind, full_sorts):
    n = 1 << 20
    r = I.stress_row(kind, 41, n)
    for k, alpha in [(n / 16, -1.0), (210.0, -0.01), (n / 2, -0.001)]:
        run = DeviceRun(r, k, alpha, L.default_params(full_sorts=full_sorts, **BRACKET), seed=5).forward()
        assert_forward_matches(run, what=f"{kind} k={k}")  # exact whether or not the bracket held


@pytest.mark.parametrize("step", [1.0 / 64, 1.0 / 4096, 2.0 ** -16])
@pytest.mark.parametrize("k,alpha", [(300.0, -0.05), (20000.0, -0.01), (150000.0, -0.5)])
def test_quantised_scores_tie_inside_the_band(step, k, alpha):
    # scores on a lattice: the band's last list holds runs of equal scores (ranked by list position in the
    # all-pairs solve, sorted in the block solve); coarse lattices reach the one-key-bucket levels
    n = 300000
    r = (np.round(I.stress_row("gaussian", 51, n) / step) * step).astype(np.float32)
    run = DeviceRun(r, k, alpha, L.default_params(**BRACKET), seed=9).forward()
    assert run.status().path == L.PATH_BRACKET
    assert_forward_matches(run, what=f"lattice {step} k={k}")


def test_bracket_path_is_bit_reproducible():
    # the band arrives in arbitrary order; fixed-point band sums and fixed-order tail sums keep b identical
    w = I.scaled(I.WORKLOADS["c5"], 4_000_000)
    r, v = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r, w.k, w.alpha, L.default_params(**BRACKET), seed=3).forward().backward(v)
    p0, b0, g0 = run.p.clone(), run.b.clone(), run.grad.clone()
    for _ in range(5):
        run.forward().backward(v)
        assert torch.equal(b0, run.b) and torch.equal(p0, run.p) and torch.equal(g0, run.grad)


@pytest.mark.parametrize("seed", [1, 2, 3])
@pytest.mark.parametrize("n,k,alpha", [(4_000_000, 3.5, -1e-5), (4_000_000, 3_999_996.5, -1e-5), (1_000_000, 2.25, -3e-6)])
def test_open_bracket_end_whose_buckets_are_one_key_wide(n, k, alpha, seed):
    # a sorted row: the strided sample never reaches the last n - K * stride scores, Eq. 8 leaves that end of the
    # bracket open, and with a tiny temperature the sample's extreme lies within 1024 keys of the bracket's other end.
    # The buckets are then one key wide, but the outermost one also holds everything beyond the sample's extreme: it
    # is not a run of equal scores and must not be solved as one.
    r = I.stress_row("sorted_ramp", 0, n)
    if k > n / 2:
        r = np.ascontiguousarray(r[:, ::-1])  # descending: the unsampled stretch is the bottom of the row
    run = DeviceRun(r, k, alpha, L.default_params(**BRACKET), seed=seed).forward()
    assert_forward_matches(run, what=f"sorted ramp n={n} k={k}")


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
@pytest.mark.parametrize("scale,alpha", [(1.0, -1e-3), (1e-20, -1e-23), (1e-20, -3e-23), (1e-30, -7e-34)])
def test_open_end_bucket_that_needs_a_second_level(scale, alpha, seed):
    # a sorted row whose last 655 scores the strided sample never sees: Eq. 8 leaves the bracket open on that side and
    # a few hundred scores lie beyond the sample's extreme, all in the outermost bucket, so a second level has to cut
    # a key range that reaches to +inf.  Its far edges lie ~1e38 away: (edge - pivot) / t overflows, and with tiny
    # scores (t ~ 1e-23) so does the low-order part of that product, which must still read as "no contribution"
    n, k = 1_002_055, 3.5
    r = (I.stress_row("sorted_ramp", 0, n).astype(np.float64) * scale).astype(np.float32)
    run = DeviceRun(r, k, alpha, L.default_params(**BRACKET), seed=seed).forward()
    st = run.status()
    assert st.a_R == float("inf") and st.fallbacks == 0
    assert_forward_matches(run, what=f"ramp x {scale} alpha={alpha} seed={seed}")


@pytest.mark.parametrize("alpha,overflows", [(-0.3, False), (-4.0, False), (-300.0, True)])
def test_half_budget_with_a_temperature_at_and_above_the_spread_of_the_scores(alpha, overflows):
    # The bracket is taken on the noised sample y = r + t e: with t above the spread of r the band in r is wider than
    # Eq. 8 predicts by the ratio of the two densities at b.  The default band buffer absorbs a factor of four (here:
    # N(0,1) scores, k = n/2, t up to 4); far beyond that every call overflows and pays the full sort, exactly, and
    # says so in the status word and the fallback counter.
    n = 1 << 20
    r = I.stress_row("gaussian", 61, n)
    ref = O.forward(r, n / 2, alpha)
    run = DeviceRun(r, n / 2, alpha, L.default_params(**BRACKET), seed=13)
    for call in range(3):
        run.forward()
        assert_forward_matches(run, ref, what=f"alpha {alpha} call {call}")
    st = run.status()
    assert st.path == L.PATH_BRACKET
    assert bool(st.status_bits & L.ST_BAND_OVERFLOW) == overflows
    assert st.fallbacks == (3 if overflows else 0)
    if not overflows:
        assert st.n_M <= band_capacity(run.ws)
