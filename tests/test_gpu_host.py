"""GPU parity, host-buffer entry point: same bits as the device-buffer calls, and the oracle's values."""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import inputs as I
from tests.gpu_util import DeviceRun, assert_backward_matches, assert_forward_matches

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n", [("c1", None), ("c2", None), ("c3", 300_001), ("c5", 2_000_000)])
@pytest.mark.parametrize("pinned", [True, False])
def test_host_step_matches_device_step(name, n, pinned):
    w = I.WORKLOADS[name] if n is None else I.scaled(I.WORKLOADS[name], n)
    if name == "c2":
        w = I.Workload("c2s", 4096, 128, w.k, w.alpha, w.seed_r, w.seed_v, w.seed_sampler, w.recipe)
        r_np, v_np = I.normal_rows_with_duplicates(w.seed_r, w.rows, w.n), I.upstream(w.seed_v, w.rows, w.n)
    else:
        r_np, v_np = I.make_scores(w), I.make_upstream(w)
    run = DeviceRun(r_np, w.k, w.alpha, None, seed=w.seed_sampler).forward().backward(v_np)
    torch.cuda.synchronize()

    def host(x):
        t = torch.from_numpy(np.ascontiguousarray(x))
        return t.pin_memory() if pinned else t

    r_h, v_h = host(r_np), host(v_np)
    p_h, g_h = host(np.zeros_like(r_np)), host(np.zeros_like(r_np))
    b_h = host(np.zeros(w.rows, np.float32))
    staging = torch.empty(4 * w.rows * w.n + w.rows, device="cuda")
    ws = L.Workspace(w.rows, w.n, None, w.seed_sampler)
    for _ in range(2):  # the second call reuses the side streams and events
        p_h.zero_(); g_h.zero_(); b_h.zero_()
        L.lapsum_forward_backward_host(r_h, v_h, w.k, w.alpha, p_h, g_h, b_h, staging, ws)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(p_h.view(w.rows, w.n), run.p.cpu()) and torch.equal(b_h, run.b.cpu())
        assert torch.equal(g_h.view(w.rows, w.n), run.grad.cpu())
    ref = assert_forward_matches(run, what=f"{name} host step")
    assert_backward_matches(run, v_np, ref.b, what=f"{name} host step")


def test_host_step_rejects_bad_arguments():
    ws = L.Workspace(2, 256, None, 1)
    h = lambda m: torch.zeros(m)
    st = torch.empty(4 * 512 + 2, device="cuda")
    with pytest.raises(ValueError):
        L.lapsum_forward_backward_host(h(512), h(512), 4.0, -0.1, h(512), h(512), h(2), st[:100], ws)
    with pytest.raises(TypeError):
        L.lapsum_forward_backward_host(h(512).cuda(), h(512), 4.0, -0.1, h(512), h(512), h(2), st, ws)
    with pytest.raises(L.LapsumError):
        L.lapsum_forward_backward_host(h(512), h(512), 4.0, 0.0, h(512), h(512), h(2), st, ws)
