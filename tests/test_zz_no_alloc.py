"""The allocation-free backward entry point, called through the C ABI.

lapsum_backward_static serves hosts that are not allowed to allocate device memory while they run (fixed memory
budget, foreign allocator, no tolerance for cudaMalloc's device synchronisation): its scratch is a fixed array
inside the library.  The check: on two calls in a row it returns what the workspace-based lapsum_backward returns,
within the gradient tolerance of the other GPU tests.  This file is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import GRAD_RTOL, to_dev

pytestmark = pytest.mark.gpu


def _reference_backward(r, v, k, alpha):
    """forward + backward through a workspace (full-sort path, so the two-kernel VJP is the one that runs)"""
    rows, n = r.shape
    ws = L.Workspace(rows, n, L.default_params(force_path=L.PATH_FULLSORT))
    p, g = torch.empty_like(r), torch.empty_like(r)
    b = torch.empty(rows, device="cuda")
    L.lapsum_forward(r, k, alpha, p, b, ws)
    L.lapsum_backward(v, r, b, k, alpha, g, ws)
    torch.cuda.synchronize()
    return b, g


@pytest.mark.parametrize("rows,n,k,alpha", [(1, 300_001, 150.0, -0.05), (3, 70_000, 4375.0, -1.0)])
def test_static_backward_matches_workspace_backward_twice(rows, n, k, alpha):
    rng = np.random.default_rng(rows * 7 + n)
    r = to_dev(rng.standard_normal((rows, n)).astype(np.float32))
    v = to_dev(rng.standard_normal((rows, n)).astype(np.float32))
    b, g_ref = _reference_backward(r, v, k, alpha)
    scale = float(g_ref.abs().max())
    assert scale > 0
    lib = L.lib()
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):  # the shared scratch keeps the previous call's contents: the second call must not care
        g = torch.full_like(r, float("nan"))
        rc = lib.lapsum_backward_static(v.data_ptr(), r.data_ptr(), b.data_ptr(), rows, n, alpha, g.data_ptr(), stream)
        assert rc == 0, L.lib().lapsum_error_string(rc)
        torch.cuda.synchronize()
        assert torch.isfinite(g).all()
        err = float((g - g_ref).abs().max()) / scale
        assert err <= GRAD_RTOL, f"call {call}: {err:.3e}"
        # different upstream on the next round, so a stale result could not pass
        v = to_dev(rng.standard_normal((rows, n)).astype(np.float32))
        _, g_ref = _reference_backward(r, v, k, alpha)
        scale = float(g_ref.abs().max())


def test_static_backward_rejects_sizes_beyond_its_limits():
    lib = L.lib()
    x = torch.zeros(8, device="cuda")
    ptr, st = x.data_ptr(), torch.cuda.current_stream().cuda_stream
    assert lib.lapsum_backward_static(ptr, ptr, ptr, 65537, 8, -1.0, ptr, st) == -2   # too many rows
    assert lib.lapsum_backward_static(ptr, ptr, ptr, 1, 1 << 30, -1.0, ptr, st) == -2
    assert lib.lapsum_backward_static(ptr, ptr, ptr, 0, 8, -1.0, ptr, st) == -2
    assert lib.lapsum_backward_static(None, ptr, ptr, 1, 8, -1.0, ptr, st) == -1
    assert lib.lapsum_backward_static(ptr, ptr, ptr, 1, 8, 0.0, ptr, st) == -4
    torch.cuda.synchronize()
