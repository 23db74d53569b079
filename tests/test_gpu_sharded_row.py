"""One row spread over several shards (dist.forward_sharded / backward_sharded) against the oracle, on ONE GPU.

The shards live in one process here, so the exchanges are plain tensor sums and concatenations; the per-shard kernels,
the exchange buffers and the merged solve are the ones a multi-GPU run uses (there the same sums are NCCL collectives;
tests/test_dist_gloo.py runs that branch between two CPU ranks).  Nothing here waits on another kernel."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import dist as D
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import B_RTOL, BUDGET_RTOL, GRAD_RTOL, P_ATOL, b_error

pytestmark = pytest.mark.gpu


def make_shards(r, cuts, params=None, seed=0):
    n = r.shape[1]
    edges = [0] + list(cuts) + [n]
    rd = torch.from_numpy(r).cuda().view(-1)
    return [L.GpuShard(rd[lo:hi].contiguous(), lo, n, params, seed) for lo, hi in zip(edges[:-1], edges[1:])]


def check(r, v, k, alpha, cuts, seed=3, params=None, expect_held=True):
    shards = make_shards(r, cuts, params, seed)
    held = D.forward_sharded(shards, k, alpha, gather_row=D.gather_row_over(shards))
    assert held == expect_held
    vd = torch.from_numpy(v).cuda().view(-1)
    v_sh = [vd[s.begin:s.begin + s.len].contiguous() for s in shards]
    D.backward_sharded(shards, v_sh, alpha)
    torch.cuda.synchronize()
    ref = O.forward(r, k, alpha)
    p = torch.cat([s.p for s in shards]).cpu().numpy().astype(np.float64)
    assert np.max(np.abs(p - ref.p[0])) <= P_ATOL
    assert abs(p.sum() - k) <= BUDGET_RTOL * k
    for s in shards:   # every shard knows the row's threshold
        assert b_error(float(s.b[0]), ref.b, r, alpha) <= B_RTOL
    g = torch.cat([s.grad for s in shards]).cpu().numpy().astype(np.float64)
    g_ref = O.backward(v, r, ref.b, alpha)[0]
    assert np.max(np.abs(g - g_ref)) <= GRAD_RTOL * np.max(np.abs(g_ref))
    gk_ref, ga_ref = O.backward_scalars(v, r, ref.b, alpha)
    for s in shards:
        assert abs(float(s.grad_k[0]) - gk_ref[0]) <= GRAD_RTOL * np.abs(v).max()
        assert abs(float(s.grad_alpha[0]) - ga_ref[0]) <= 10 * GRAD_RTOL * max(abs(ga_ref[0]), 1e-3 * np.abs(v).max() * k / abs(alpha))
    return shards


@pytest.mark.parametrize("cuts", [[], [1_500_000], [700_001, 2_222_222], [4, 2_999_990]])
@pytest.mark.parametrize("alpha", [-0.02, 0.05])
def test_sharded_row_matches_the_oracle(cuts, alpha):
    w = I.scaled(I.WORKLOADS["c4"], 3_000_000)
    r, v = I.make_scores(w), I.make_upstream(w)
    shards = check(r, v, w.k, alpha, cuts, seed=w.seed_sampler)
    # sample, bracket ends and band counts are those of the unsharded row, bit for bit
    k_eff = w.k if alpha < 0 else w.n - w.k
    want = O.bracket(r, k_eff, -abs(alpha), 5.16, w.seed_sampler)
    sts = [s.ws.status() for s in shards]
    for st in sts:   # every shard derived the same bracket from the merged sample
        assert np.float32(st.a_L).view(np.uint32) == np.float32(want.a_L).view(np.uint32)
        assert np.float32(st.a_R).view(np.uint32) == np.float32(want.a_R).view(np.uint32)
    # the shards' own counts (what each stream pass recorded) add up to the row's
    assert sum(st.n_M for st in sts) == want.n_M and sum(st.n_R for st in sts) == want.n_R


def test_sharded_row_agrees_with_the_single_gpu_forward():
    w = I.scaled(I.WORKLOADS["c5"], 5_000_000)
    r = I.make_scores(w)
    shards = make_shards(r, [1_000_000, 2_500_000, 4_999_999], seed=w.seed_sampler)
    assert D.forward_sharded(shards, w.k, w.alpha)
    rd = torch.from_numpy(r).cuda()
    ws = L.Workspace(1, w.n, None, w.seed_sampler)
    p, b = torch.empty_like(rd), torch.empty(1, device="cuda")
    L.lapsum_forward(rd, w.k, w.alpha, p, b, ws)
    torch.cuda.synchronize()
    # the same sample, bracket and band; the tails are summed in another grouping, so the last bits of b may differ
    assert abs(float(b[0]) - float(shards[0].b[0])) <= 1e-6 * abs(float(b[0]))
    assert float((torch.cat([s.p for s in shards]) - p.view(-1)).abs().max()) <= 5e-7


def test_failed_certificate_gathers_the_row():
    # a bracket of half a standard deviation misses about two times in three: the sharded solve must say so (NaN
    # threshold) and the orchestrator must end with the ordinary forward of the gathered row
    n, k, alpha = 400_000, 300.0, -0.05
    r = I.stress_row("gaussian", 5, n)
    v = I.upstream(6, 1, n)
    outcomes = set()
    for seed in range(10):
        shards = make_shards(r, [133_333, 266_667], L.default_params(z=0.5), seed)
        held = D.forward_sharded(shards, k, alpha, gather_row=D.gather_row_over(shards))
        outcomes.add(held)
        torch.cuda.synchronize()
        ref = O.forward(r, k, alpha)
        p = torch.cat([s.p for s in shards]).cpu().numpy().astype(np.float64)
        assert np.max(np.abs(p - ref.p[0])) <= P_ATOL
        assert b_error(float(shards[1].b[0]), ref.b, r, alpha) <= B_RTOL
    assert outcomes == {True, False}


def test_shard_calls_check_their_arguments():
    lib = L.lib()
    shards = make_shards(I.stress_row("gaussian", 1, 50_000), [20_000])
    ws = shards[0].ws
    st = torch.cuda.current_stream().cuda_stream
    rp = shards[0].r.data_ptr()
    assert lib.lapsum_shard_sample(rp, 40_000, 20_000, 50_000, -0.1, ws.ptr, st) == -2      # shard beyond the row
    assert lib.lapsum_shard_sample(rp, 0, 20_000, 60_000, -0.1, ws.ptr, st) == -5           # another row length
    assert lib.lapsum_shard_stream(rp, 20_000, 50_000, 0.0, -0.1, ws.ptr, st) == -3
    assert lib.lapsum_shard_solve(50_000, 5.0, 0.0, shards[0].b.data_ptr(), ws.ptr, st) == -4
    plain = L.Workspace(1, 50_000)
    assert lib.lapsum_shard_sample(rp, 0, 20_000, 50_000, -0.1, plain.ptr, st) == -8         # not a shard workspace
    torch.cuda.synchronize()
