"""Helpers of the GPU parity tests: run the CUDA path through the C ABI binding and compare with the oracle.

Tolerances (fp32 path against the fp64 oracle on the same seeded inputs):
  p      2e-6 absolute
  b      1e-5 relative to max(|b|, half the range of the row's scores, |alpha|): the threshold moves with the scores
         (shift invariance), so their spread, not 1, is the scale of a threshold near zero
  budget |sum p - k| <= 1e-4 k
  grad   1e-4 of the oracle gradient's max-norm
  sorted keys, payload indices, bracket ends and band counts: bit-exact
"""
import numpy as np
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O

P_ATOL = 2e-6
B_RTOL = 1e-5
BUDGET_RTOL = 1e-4
GRAD_RTOL = 1e-4


def b_scale(b_ref, r, alpha):
    """Per row: the magnitude |b - b_oracle| is measured against.  b is an input value plus an offset of at most the gap
    to the next score, both rounded in fp32, so its error scales with max(|b|, spread of the scores); |alpha| covers
    rows of one score (their offset is a multiple of the temperature)."""
    r = np.asarray(r, dtype=np.float64).reshape(len(np.atleast_1d(b_ref)), -1)
    half_range = 0.5 * (r.max(axis=1) - r.min(axis=1))
    return np.maximum(np.maximum(np.abs(np.atleast_1d(b_ref)), half_range), abs(alpha))


def b_error(b, b_ref, r, alpha):
    """max over rows of |b - b_oracle| / b_scale"""
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.max(np.abs(b - np.atleast_1d(b_ref)) / b_scale(b_ref, r, alpha)))


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class DeviceRun:
    def __init__(self, r, k, alpha, params=None, seed=0):
        r = np.ascontiguousarray(r, dtype=np.float32)
        if r.ndim == 1:
            r = r.reshape(1, -1)
        self.r_np = r
        self.rows, self.n = r.shape
        self.k, self.alpha = float(k), float(alpha)
        self.ws = L.Workspace(self.rows, self.n, params, seed)
        self.r = to_dev(r)
        self.p = torch.full_like(self.r, float("nan"))
        self.b = torch.full((self.rows,), float("nan"), device="cuda")

    def forward(self):
        L.lapsum_forward(self.r, self.k, self.alpha, self.p, self.b, self.ws)
        torch.cuda.synchronize()
        return self

    def backward(self, v):
        self.v = to_dev(np.ascontiguousarray(v, dtype=np.float32).reshape(self.rows, self.n))
        self.grad = torch.full_like(self.r, float("nan"))
        L.lapsum_backward(self.v, self.r, self.b, self.k, self.alpha, self.grad, self.ws)
        torch.cuda.synchronize()
        return self

    def status(self):
        return self.ws.status()


def assert_forward_matches(run: DeviceRun, ref=None, what=""):
    if ref is None:
        ref = O.forward(run.r_np, run.k, run.alpha)
    p = run.p.cpu().numpy().astype(np.float64)
    b = run.b.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(p)) and np.all(np.isfinite(b)), what
    err_p = float(np.max(np.abs(p - ref.p)))
    assert err_p <= P_ATOL, f"{what}: max|p - p_oracle| = {err_p:.3e}"
    err_b = b_error(b, ref.b, run.r_np, run.alpha)
    assert err_b <= B_RTOL, f"{what}: b rel err {err_b:.3e}"
    budget = np.abs(run.p.double().sum(dim=1).cpu().numpy() - run.k)
    assert float(budget.max()) <= BUDGET_RTOL * run.k, f"{what}: |sum p - k| = {float(budget.max()):.3e}"
    assert float(p.min()) >= 0.0 and float(p.max()) <= 1.0
    return ref


def assert_backward_matches(run: DeviceRun, v, ref_b, what=""):
    g_ref = O.backward(v, run.r_np, ref_b, run.alpha)
    g = run.grad.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(g)), what
    # max-norm of the oracle gradient, floored for rows whose gradient cancels (n = 1, constant v):
    # there the natural scale is max f * max|v|
    t = abs(run.alpha)
    f = np.exp(-np.abs(np.asarray(ref_b, np.float64).reshape(-1, 1) - run.r_np.astype(np.float64)) / t) / (2 * t)
    floor = 0.01 * f.max(axis=1, keepdims=True) * np.abs(v).max(axis=1, keepdims=True).astype(np.float64)
    scale = np.maximum(np.max(np.abs(g_ref), axis=1, keepdims=True), floor)
    scale = np.maximum(scale, 1e-30)  # an fp32 gradient cannot hold values below ~1e-38 (plateaus with tiny t)
    err = float(np.max(np.abs(g - g_ref) / scale))
    assert err <= GRAD_RTOL, f"{what}: grad err / max-norm = {err:.3e}"
    return g_ref
