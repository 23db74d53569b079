"""The C-ABI library loads on a CPU-only box and exports every symbol include/lapsum.h declares.
Only host-side entry points are called here (sizing and argument checks); nothing touches a GPU."""
import ctypes as C
import os
import re

import pytest

import paper_2608_06912_b200 as L
from paper_2608_06912_b200 import binding

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "lapsum.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lapsum_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert len(names) >= 12
    lib = L.lib()
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(binding.EXPORTS)


def test_defaults():
    p = L.default_params()
    assert p.z == pytest.approx(5.16) and p.force_path == L.PATH_AUTO and p.block_max_n == 16384
    assert p.bracket_min_n == 16385 and p.sort_payload == 0


def test_workspace_sizing_is_host_only_and_monotone():
    small = L.lapsum_workspace_bytes(4, 4096)
    mid = L.lapsum_workspace_bytes(1, 1 << 20)
    big = L.lapsum_workspace_bytes(1, 10**8)
    assert 0 < small < mid < big
    # bracket path at 1e8: two key buffers for the full-sort fallback dominate (2 x 400 MB)
    assert 8e8 < big < 1.0e9
    with_payload = L.lapsum_workspace_bytes(1, 1 << 20, L.default_params(sort_payload=1))
    assert with_payload >= mid + 2 * 4 * (1 << 20)


def test_argument_errors_are_reported_before_any_device_work():
    lib = L.lib()
    out = C.c_size_t()
    assert lib.lapsum_workspace_bytes(0, 10, None, C.byref(out)) == -2
    assert lib.lapsum_workspace_bytes(1, 1 << 30, None, C.byref(out)) == -2
    assert lib.lapsum_workspace_bytes(1, (1 << 30) - 1, None, C.byref(out)) == 0
    assert lib.lapsum_workspace_bytes(1, 10, None, None) == -1
    bad = L.default_params(force_path=L.PATH_BLOCK)
    assert lib.lapsum_workspace_bytes(1, 100000, C.byref(bad), C.byref(out)) == -7
    bad = L.default_params(force_path=L.PATH_BRACKET)
    assert lib.lapsum_workspace_bytes(1, 1000, C.byref(bad), C.byref(out)) == -7
    bad = L.default_params(z=-1.0)
    assert lib.lapsum_workspace_bytes(1, 1000, C.byref(bad), C.byref(out)) == -7
    # forward / backward: null pointers, bad budget, bad alpha, unknown workspace
    assert lib.lapsum_forward(None, 1, 8, 2.0, -1.0, None, None, None, None) == -1
    fake = 4096
    assert lib.lapsum_forward(fake, 1, 8, 0.0, -1.0, fake, fake, fake, None) == -3
    assert lib.lapsum_forward(fake, 1, 8, 8.0, -1.0, fake, fake, fake, None) == -3
    assert lib.lapsum_forward(fake, 1, 8, 2.0, 0.0, fake, fake, fake, None) == -4
    assert lib.lapsum_forward(fake, 1, 8, 2.0, float("nan"), fake, fake, fake, None) == -4
    assert lib.lapsum_forward(fake, 1, 8, 2.0, 1.0, fake, fake, fake, None) == -5  # alpha > 0 is a valid problem
    assert lib.lapsum_forward(fake, 1, 8, 2.0, -1.0, fake, fake, fake, None) == -5
    assert lib.lapsum_backward(fake, fake, fake, 2.0, -1.0, fake, fake, None) == -5
    assert lib.lapsum_workspace_release(fake) == -5
    assert lib.lapsum_forward_row_budgets(fake, 1, 8, None, -1.0, fake, fake, fake, None) == -1
    assert lib.lapsum_forward_row_budgets(fake, 1, 8, fake, 0.0, fake, fake, fake, None) == -4
    assert lib.lapsum_forward_row_budgets(fake, 1, 8, fake, -1.0, fake, fake, fake, None) == -5
    assert lib.lapsum_error_string(-3).decode().startswith("budget")
    assert lib.lapsum_launch_count() == 0


def test_binding_refuses_to_run_without_a_gpu():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        L.Workspace(1, 128)


def test_dispatch_rules_without_a_gpu():
    d = L.lapsum_describe
    assert d(65536, 128).path == L.PATH_BLOCK          # routing shape: short rows
    assert d(4, 4096).path == L.PATH_BLOCK
    assert d(8, 16384).path == L.PATH_BLOCK            # a batch keeps the block path up to its limit
    assert d(1, 8192).path == L.PATH_BLOCK
    assert d(1, 8193).path == L.PATH_BRACKET           # a single long row is faster on the bracket path
    assert d(2, 16385).path == L.PATH_BRACKET          # every row longer than the block path
    assert d(1, 10**8).path == L.PATH_BRACKET
    assert d(1, 10**6, params=L.default_params(force_path=L.PATH_FULLSORT)).path == L.PATH_FULLSORT
    # a caller that raises bracket_min_n gets the full sort in between, and no early bracket for single rows
    p = L.default_params(bracket_min_n=10**6)
    assert d(1, 16000, params=p).path == L.PATH_BLOCK and d(1, 200000, params=p).path == L.PATH_FULLSORT
    with pytest.raises(L.LapsumError):
        d(1, 4095, params=L.default_params(force_path=L.PATH_BRACKET))   # below the bracket path's floor
    with pytest.raises(L.LapsumError):
        d(1, 20000, params=L.default_params(force_path=L.PATH_BLOCK))    # above the block path's limit
    with pytest.raises(L.LapsumError):
        d(1, 1000, k=1000.0)                                             # k must be below n


@pytest.mark.parametrize("n,k,K,j,l", [
    # the two long-row configurations and the megapixel shape, evaluated by hand from Eq. 8 with z = 5.16
    (10**7, 2000.0, 46416, 46390, 46423), (10**8, 20000.0, 215444, 215367, 215435), (1 << 20, 210.0, 10322, 10312, 10328),
    (10**8, 10**8 / 16, 215444, 201398, 202559),
])
def test_sample_size_and_ranks_of_the_library_match_hand_values_and_the_oracle(n, k, K, j, l):
    from oracle import lapsum_oracle as O
    plan = L.lapsum_describe(1, n, k)
    assert (plan.K, plan.j, plan.l) == (K, j, l)
    assert plan.stride == n // K and plan.band_capacity >= 8192
    assert O.sample_count(n) == K and tuple(O.bracket_indices(n, k, 5.16))[-2:] == (j, l)


def test_temperatures_that_fp32_cannot_hold_are_rejected_on_the_host():
    fake = C.c_void_p(256)  # never dereferenced: the argument check returns first
    for alpha in (0.0, 1e-39, -1e-39, -1e-300, -1e39, 1e39, float("nan"), float("-inf"), float("inf")):
        assert L.lib().lapsum_forward(fake, 1, 8, 2.0, alpha, fake, fake, fake, None) == -4, alpha
    assert L.lib().lapsum_forward(fake, 1, 8, 9.0, -0.1, fake, fake, fake, None) == -3   # k >= n
    assert L.lib().lapsum_forward(fake, 1, 8, 2.0, -1.2e-38, fake, fake, fake, None) == -5  # valid problem, unknown workspace


def test_workspace_of_a_batch_of_long_rows_has_up_to_sixteen_slots():
    one = L.lapsum_workspace_bytes(1, 1 << 20)
    # the per-row threshold pairs (8 bytes a row) and parameter sets (72 bytes a row), 256-byte aligned, are part of every slot
    for rows, slots in ((2, 2), (4, 4), (9, 9), (40, 16)):
        got = L.lapsum_workspace_bytes(rows, 1 << 20)
        assert slots * one <= got <= slots * (one + 256 * (1 + rows // 32) + 256 * (1 + rows * 72 // 256)), (rows, got, one)
    # short rows are one launch for the whole batch: no slots
    assert L.lapsum_workspace_bytes(9, 4096) < 2 * L.lapsum_workspace_bytes(1, 4096) + 9 * 4096
    # very long rows: one slot only (a single row's buffers already exceed the 8 GB at which slots are given up)
    assert L.lapsum_workspace_bytes(1, 10**9) <= L.lapsum_workspace_bytes(4, 10**9) < L.lapsum_workspace_bytes(1, 10**9) + 4096 < 9e9


def test_host_checks_apply_to_the_scalars_in_use_only():
    lib = L.lib()
    fake = 4096
    # k is replaced by a vector: its scalar is not looked at; alpha is in use and must be valid
    assert lib.lapsum_forward_rows(fake, 1, 8, fake, None, -5.0, 0.0, fake, fake, fake, None) == -4
    assert lib.lapsum_forward_rows(fake, 1, 8, fake, None, -5.0, -1.0, fake, fake, fake, None) == -5
    assert lib.lapsum_forward_rows(fake, 1, 8, None, fake, 9.0, 0.0, fake, fake, fake, None) == -3
    assert lib.lapsum_forward_rows(fake, 1, 8, None, fake, 2.0, 0.0, fake, fake, fake, None) == -5
    assert lib.lapsum_backward_rows(fake, fake, fake, fake, 0.0, fake, None, None, fake, None) == -5
    assert lib.lapsum_backward_rows(fake, fake, fake, None, 0.0, fake, None, None, fake, None) == -4
