"""The allocation-free backward entry point, called through the C ABI.

lapsum_backward_static serves hosts that are not allowed to allocate device memory while they run (fixed memory
budget, foreign allocator, no tolerance for cudaMalloc's device synchronisation): its scratch is a fixed array
inside the library.  The checks: on two calls in a row it returns the gradient of the CPU oracle (Eq. 5) within the
gradient tolerance of the other GPU tests, it agrees with the workspace-based lapsum_backward, and the device's free
memory is the same after the calls as before them.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from tests.gpu_util import B_RTOL, GRAD_RTOL, b_error, to_dev

pytestmark = pytest.mark.gpu


def _workspace_forward_backward(r, v, k, alpha):
    """forward + backward through a workspace (full-sort path, so the two-kernel VJP is the one that runs)"""
    rows, n = r.shape
    ws = L.Workspace(rows, n, L.default_params(force_path=L.PATH_FULLSORT))
    p, g = torch.empty_like(r), torch.empty_like(r)
    b = torch.empty(rows, device="cuda")
    L.lapsum_forward(r, k, alpha, p, b, ws)
    L.lapsum_backward(v, r, b, k, alpha, g, ws)
    torch.cuda.synchronize()
    ws.release()
    return b, g


def _scores(rows, n, seed):
    rng = np.random.default_rng(seed)
    r = rng.standard_normal((rows, n)).astype(np.float32)
    r += np.arange(rows, dtype=np.float32)[:, None] * 0.75   # every row has its own threshold
    return r, rng


@pytest.mark.parametrize("rows,n,k,alpha", [
    (1, 300_001, 150.0, -0.05),     # one long row, odd length
    (3, 70_000, 4375.0, -1.0),      # rows that differ in b
    (3, 70_001, 300.0, -0.2),       # rows that are not 16-byte aligned: the kernels' scalar path
    (2, 100_000, 99_000.0, 0.5),    # alpha > 0: the gradient changes sign
])
def test_static_backward_matches_the_oracle_twice_and_allocates_nothing(rows, n, k, alpha):
    r_np, rng = _scores(rows, n, rows * 7 + n)
    r = to_dev(r_np)
    ref = O.forward(r_np, k, alpha, want_p=False)
    assert rows == 1 or np.ptp(ref.b) > 0.5
    lib = L.lib()
    stream = torch.cuda.current_stream().cuda_stream
    v_np = [rng.standard_normal((rows, n)).astype(np.float32) for _ in range(2)]  # another upstream on the second call,
    v = [to_dev(x) for x in v_np]                                                 # so a stale result could not pass
    ws_out = [_workspace_forward_backward(r, x, k, alpha) for x in v]
    b = ws_out[0][0]
    assert b_error(b.cpu().numpy(), ref.b, r_np, alpha) <= B_RTOL
    g = [torch.full_like(r, float("nan")) for _ in range(2)]
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for call in range(2):  # the shared scratch keeps the previous call's contents: the second call must not care
        rc = lib.lapsum_backward_static(v[call].data_ptr(), r.data_ptr(), b.data_ptr(), rows, n, alpha,
                                        g[call].data_ptr(), stream)
        assert rc == 0, lib.lapsum_error_string(rc)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the entry point must not allocate device memory"
    for call in range(2):
        got = g[call].cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        want = O.backward(v_np[call], r_np, ref.b, alpha)
        scale = np.max(np.abs(want), axis=1, keepdims=True)
        assert np.all(scale > 0)
        err = float(np.max(np.abs(got - want) / scale))
        assert err <= GRAD_RTOL, f"call {call}: against the oracle {err:.3e}"
        g_ws = ws_out[call][1]
        err_ws = float((g[call] - g_ws).abs().max() / g_ws.abs().max())
        assert err_ws <= GRAD_RTOL, f"call {call}: against the workspace backward {err_ws:.3e}"


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
