"""GPU parity of the 16-bit storage types (lapsum_params.io_dtype = fp16 / bf16; lapsum_forward_io, lapsum_backward_io).

Scores and upstream gradients are drawn as usual and rounded to the storage type; the oracle gets the very same values
up-converted (exact in fp32), so it needs no new arithmetic.  The arithmetic of the CUDA path stays fp32, hence:
  b            1e-5 relative, as for fp32 storage
  p            the oracle's mask rounded to the storage type, +- one ulp of that type, + the fp32 budget 2e-6
  |sum p - k|  1e-4 k + (eps / 2) k: every stored p_i is off by at most half an ulp, eps = 2^-10 (fp16), 2^-7 (bf16)
  grad         1e-4 of the max-norm + half an ulp of the storage type at the value
  sample values, bracket ends, band counts: bit-exact (they never leave fp32)
"""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import B_RTOL, BUDGET_RTOL, GRAD_RTOL, P_ATOL, b_error

pytestmark = pytest.mark.gpu

EPS = {L.IO_F16: 2.0 ** -10, L.IO_BF16: 2.0 ** -7}     # spacing of the type relative to the value (one ulp at 1.0)
TINY = {L.IO_F16: 2.0 ** -24, L.IO_BF16: 2.0 ** -133}   # smallest subnormal


def to_storage(x, io):
    """round an fp32 numpy array to the storage type; returns the torch tensor (CUDA) and the values as float32 numpy"""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(L.IO_TORCH[io]).cuda()
    return t, t.float().cpu().numpy()


def ulp(x, io):
    """one unit in the last place of the storage type at |x| (float64 numpy)"""
    ax = np.abs(x)
    e = np.floor(np.log2(np.maximum(ax, 1e-300)))
    return np.maximum(2.0 ** e * EPS[io], TINY[io])


def run_and_check(r32, v32, k, alpha, io, params=None, seed=3, what="", allow_bits=0):
    rows, n = r32.shape
    prm = L.default_params(io_dtype=io, **(params or {}))
    ws = L.Workspace(rows, n, prm, seed)
    r, r_np = to_storage(r32, io)
    v, v_np = to_storage(v32, io)
    p, g = torch.empty_like(r), torch.empty_like(r)
    b = torch.empty(rows, device="cuda")
    gk, ga = torch.empty(rows, device="cuda"), torch.empty(rows, device="cuda")
    L.lapsum_forward_io(r, None, None, k, alpha, p, b, ws)
    L.lapsum_backward_io(v, r, b, None, alpha, g, gk, ga, ws)
    torch.cuda.synchronize()
    st = ws.status()
    assert not (st.status_bits & ~allow_bits), hex(st.status_bits)
    ref = O.forward(r_np, k, alpha)
    bg = b.cpu().numpy().astype(np.float64)
    assert b_error(bg, ref.b, r_np, alpha) <= B_RTOL, what
    pg = p.float().cpu().numpy().astype(np.float64)
    p_ref_T = torch.from_numpy(ref.p.astype(np.float32)).to(L.IO_TORCH[io]).float().numpy().astype(np.float64)
    assert np.all(np.abs(pg - p_ref_T) <= ulp(p_ref_T, io) + P_ATOL), f"{what}: mask beyond one ulp of the storage type"
    assert np.all(np.abs(pg.sum(axis=1) - k) <= (BUDGET_RTOL + EPS[io] / 2) * k), what
    assert pg.min() >= 0.0 and pg.max() <= 1.0
    g_ref = O.backward(v_np, r_np, ref.b, alpha)
    gg = g.float().cpu().numpy().astype(np.float64)
    # max-norm of the oracle gradient, floored for rows whose gradient cancels (n = 1): the natural scale is max f * max|v|
    t = abs(alpha)
    f = np.exp(-np.abs(ref.b.reshape(-1, 1) - r_np.astype(np.float64)) / t) / (2 * t)
    floor = 0.01 * f.max(axis=1, keepdims=True) * np.abs(v_np).max(axis=1, keepdims=True).astype(np.float64)
    scale = np.maximum(np.maximum(np.max(np.abs(g_ref), axis=1, keepdims=True), floor), 1e-30)
    assert np.all(np.abs(gg - g_ref) <= GRAD_RTOL * scale + ulp(g_ref, io) / 2 * 1.01), what
    gk_ref, _ = O.backward_scalars(v_np, r_np, ref.b, alpha)
    assert np.max(np.abs(gk.cpu().numpy() - gk_ref)) <= GRAD_RTOL * np.abs(v_np).max(), what
    return ws, st, r_np, ref


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
@pytest.mark.parametrize("name,rows", [("c1", None), ("c2", 4096)])
def test_short_row_configs(name, rows, io):
    w = I.WORKLOADS[name]
    r, v = I.make_scores(w), I.make_upstream(w)
    if rows:
        r, v = r[:rows], v[:rows]
    ws, st, _, _ = run_and_check(r, v, w.k, w.alpha, io, what=f"{name} {L.IO_NAMES[io]}")
    assert st.path == L.PATH_BLOCK


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
@pytest.mark.parametrize("rows,n,k,alpha", [(3, 1, 0.3, -0.5), (7, 5, 2.0, -0.05), (9, 100, 7.5, -0.3), (4, 129, 64.0, -0.02),
                                            (3, 1000, 62.5, -1.0), (2, 4097, 256.0, 0.05), (2, 16384, 100.0, -0.01),
                                            (300, 700, 30.0, -0.05), (20, 8192, 512.0, -1.0)])
def test_block_path_shapes(rows, n, k, alpha, io):
    rng = np.random.default_rng(rows * 1000 + n)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    v = rng.standard_normal((rows, n)).astype(np.float32)
    run_and_check(r, v, k, alpha, io, what=f"{rows}x{n}")


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
@pytest.mark.parametrize("name,n", [("c3", 1 << 20), ("c4", 10_000_000), ("c5", 3_000_001), ("paper1e6", 10**6)])
def test_long_row_configs_on_the_bracket_path(name, n, io):
    w = I.WORKLOADS[name]
    if n != w.n:
        w = I.scaled(w, n)
    r, v = I.make_scores(w), I.make_upstream(w)
    ws, st, r_np, ref = run_and_check(r, v, w.k, w.alpha, io, seed=w.seed_sampler, what=f"{w.name} {L.IO_NAMES[io]}")
    assert st.path == L.PATH_BRACKET and st.fallbacks == 0
    # sample, bracket and band counts never leave fp32: bit-exact against the oracle's bracket on the same values
    want = O.bracket(r_np, w.k, w.alpha, 5.16, w.seed_sampler)
    assert (st.K, st.j, st.l) == (want.K, want.j, want.l)
    assert np.float32(st.a_L).view(np.uint32) == np.float32(want.a_L).view(np.uint32)
    assert np.float32(st.a_R).view(np.uint32) == np.float32(want.a_R).view(np.uint32)
    assert (st.n_L, st.n_M, st.n_R) == (want.n_L, want.n_M, want.n_R)


def test_c5_at_full_size_with_bf16_storage():
    # the 16-bit bench row (bench.py --config c5 --dtype bf16) in the launch configuration the bench times
    test_long_row_configs_on_the_bracket_path("c5", I.WORKLOADS["c5"].n, L.IO_BF16)


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
@pytest.mark.parametrize("params", [dict(force_path=L.PATH_FULLSORT), dict(force_path=L.PATH_BRACKET, full_sorts=1),
                                    dict(force_path=L.PATH_FULLSORT, sort_payload=1)])
@pytest.mark.parametrize("n,k,alpha", [(16385, 100.0, -0.05), (100003, 6250.0, -1.0), (1 << 20, 210.0, -0.01)])
def test_full_sort_and_sorted_bracket_modes(n, k, alpha, params, io):
    rng = np.random.default_rng(n)
    r = rng.standard_normal((1, n)).astype(np.float32)
    v = rng.standard_normal((1, n)).astype(np.float32)
    run_and_check(r, v, k, alpha, io, params, what=f"n={n} {params}")


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
def test_forced_fallback_and_widening_with_16_bit_scores(io):
    # a narrow z makes the sampled bracket miss now and then: the device-launched widened attempt and, with no widening
    # allowed, the device-launched full sort both have to read the 16-bit row
    n, k, alpha = 500_000, 400.0, -0.05
    r = I.stress_row("gaussian", 21, n)
    v = I.upstream(22, 1, n)
    seen = {"widened": 0, "fallback": 0}
    for seed in range(12):
        for mw in (2, 0):
            ws, st, _, _ = run_and_check(r, v, k, alpha, io, dict(z=0.7, max_widenings=mw, force_path=L.PATH_BRACKET),
                                         seed=seed, what=f"z=0.7 seed {seed}",
                                         allow_bits=L.ST_WIDENED | L.ST_ROOT_LEFT | L.ST_ROOT_RIGHT | L.ST_FALLBACK)
            seen["widened"] += st.widenings
            seen["fallback"] += st.fallbacks
    assert seen["widened"] >= 1 and seen["fallback"] >= 1


@pytest.mark.parametrize("io", [L.IO_F16, L.IO_BF16])
def test_rows_with_their_own_parameters_in_16_bit(io):
    rng = np.random.default_rng(5)
    for rows, n in [(40, 100), (6, 3000), (2, 50_000)]:
        r32 = rng.standard_normal((rows, n)).astype(np.float32)
        k = rng.uniform(1.0, n / 4, rows)
        alpha = -(10.0 ** rng.uniform(-1.5, 0.0, rows))
        alpha[::3] *= -1
        ws = L.Workspace(rows, n, L.default_params(io_dtype=io), 2)
        r, r_np = to_storage(r32, io)
        p, b = torch.empty_like(r), torch.empty(rows, device="cuda")
        L.lapsum_forward_io(r, torch.from_numpy(k).cuda(), torch.from_numpy(alpha).cuda(), 1.0, -1.0, p, b, ws)
        torch.cuda.synchronize()
        assert ws.status().status_bits == 0
        pg = p.float().cpu().numpy().astype(np.float64)
        for i in range(rows):
            ref = O.forward(r_np[i], k[i], alpha[i])
            assert b_error(float(b[i]), ref.b, r_np[i], alpha[i]) <= B_RTOL
            pr = torch.from_numpy(ref.p[0].astype(np.float32)).to(L.IO_TORCH[io]).float().numpy().astype(np.float64)
            assert np.all(np.abs(pg[i] - pr) <= ulp(pr, io) + P_ATOL)


def test_entry_points_and_workspaces_must_agree_on_the_type():
    ws16 = L.Workspace(2, 256, L.default_params(io_dtype=L.IO_BF16))
    ws32 = L.Workspace(2, 256)
    r32 = torch.zeros(2, 256, device="cuda")
    b = torch.empty(2, device="cuda")
    with pytest.raises(L.LapsumError) as e:
        L.lapsum_forward(r32, 4.0, -1.0, torch.empty_like(r32), b, ws16)     # float entry point, bf16 workspace
    assert e.value.code == -5
    with pytest.raises(TypeError):
        L.lapsum_forward_io(r32, None, None, 4.0, -1.0, torch.empty_like(r32), b, ws16)
    L.lapsum_forward_io(r32, None, None, 4.0, -1.0, torch.empty_like(r32), b, ws32)  # fp32 through the typed entry point
    torch.cuda.synchronize()
    with pytest.raises(L.LapsumError):
        L.Workspace(2, 256, L.default_params(io_dtype=7))
