"""A forward + backward captured into a CUDA graph and replayed gives the results of the direct calls, on every path
(the long-row paths launch their repairs from the device and clear their control block behind themselves, so a replay
needs nothing from the host), and a replay sees new contents of the same input buffers."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from tests.gpu_util import GRAD_RTOL, P_ATOL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,n,k,alpha,params", [
    (300, 100, 7.0, -0.1, {}),                 # 16 lanes per row
    (6, 4096, 64.0, -0.05, {}),                # cluster of blocks per row
    (1, 300_001, 500.0, -0.02, {}),            # bracket path
    (1, 300_001, 500.0, -0.02, dict(band_capacity=64)),   # every call overflows: the device launches the full sort
    (5, 40_001, 80.0, -0.05, {}),              # a group of long rows
    (1, 200_000, 300.0, 0.03, dict(force_path=L.PATH_FULLSORT)),
])
def test_replay_equals_direct_calls(rows, n, k, alpha, params):
    rng = np.random.default_rng(rows + n)
    r_np = [rng.standard_normal((rows, n)).astype(np.float32) for _ in range(2)]
    v_np = rng.standard_normal((rows, n)).astype(np.float32)
    r, v = torch.from_numpy(r_np[0]).cuda(), torch.from_numpy(v_np).cuda()
    ws = L.Workspace(rows, n, L.default_params(**params), 7)
    p, g, b = torch.empty_like(r), torch.empty_like(r), torch.empty(rows, device="cuda")
    side = torch.cuda.Stream()

    def step(stream):
        L.lapsum_forward(r, k, alpha, p, b, ws, stream)
        L.lapsum_backward(v, r, b, k, alpha, g, ws, stream)

    with torch.cuda.stream(side):
        step(side)                              # the workspace has served a call before it is captured
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    for which in (0, 1, 0):                     # new scores in the same buffer between replays
        r.copy_(torch.from_numpy(r_np[which]))
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            step(side)
        torch.cuda.synchronize()
        want = (p.clone(), g.clone(), b.clone())
        p.zero_(); g.zero_(); b.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(p, want[0]) and torch.equal(g, want[1]) and torch.equal(b, want[2])
    ref = O.forward(r_np[0], k, alpha)
    assert np.max(np.abs(p.cpu().numpy().astype(np.float64) - ref.p)) <= P_ATOL
    g_ref = O.backward(v_np, r_np[0], ref.b, alpha)
    assert np.max(np.abs(g.cpu().numpy().astype(np.float64) - g_ref) / np.max(np.abs(g_ref), axis=1, keepdims=True)) <= GRAD_RTOL
    st = ws.status()
    if params.get("band_capacity") == 64:
        assert st.fallbacks >= 7 and st.status_bits & L.ST_BAND_OVERFLOW
