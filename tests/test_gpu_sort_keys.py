"""Sorted keys of the kernels the forward itself sorts with, bit for bit against the oracle's stable sort
(App. A "after sorting").

lapsum_debug_sort_pairs with idx_out = NULL launches the forward's own kernel for the shape, in the forward's own
launch configuration, and has it write the row as its sort left it: the one-warp-per-row shuffle network (n <= 128),
the register bitonic network of the block kernel at every number of keys per thread (2, 4, 8, 16; both the thread
counts used with fewer rows than SMs and with more), the cluster network over 4 and over 8 blocks, and the keys-only
radix chain of the long-row paths.  Rows carry heavy ties, +0 / -0, denormals and ragged lengths.
"""
import numpy as np
import pytest
import torch

import paper_2608_06912_b200 as L
from oracle import lapsum_oracle as O
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


def rows_with_ties(rows, n, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, n)).astype(np.float32)
    if n > 8:
        x[:, rng.integers(0, n, n // 3)] = x[:, [0]]            # a third of every row equals its first score
        lv = rng.integers(0, n, n // 4)
        x[:, lv] = np.round(x[:, lv] * 4) / 4                    # a lattice of further ties
        x[:, 1], x[:, 2] = 0.0, -0.0
        x[:, 3], x[:, 4] = 1e-41, -1e-41                         # denormals of both signs
        x[:, 5] = np.float32(-3.0e38)
        x[:, 6] = np.float32(3.0e38)
    return x


def sorted_keys_from_the_library(x, params=None):
    rows, n = x.shape
    ws = L.Workspace(rows, n, params)
    out = torch.full((rows, n), float("nan"), device="cuda", dtype=torch.float32)
    L.lapsum_debug_sort_pairs(to_dev(x), out, None, ws)
    torch.cuda.synchronize()
    st = ws.status()
    assert st.lookback_timeouts == 0
    return out.cpu().numpy(), ws


def assert_rows_bit_exact(got, x):
    for row in range(x.shape[0]):
        want, _ = O.sort_pairs(x[row])
        assert np.array_equal(got[row].view(np.uint32), want.view(np.uint32)), f"row {row}"


@pytest.mark.parametrize("rows,n", [(5, 1), (5, 7), (16, 32), (1003, 33), (1003, 64), (1003, 100), (16, 128), (1003, 128)])
def test_warp_kernels_sorted_keys(rows, n):
    x = rows_with_ties(rows, n, 10 + n)
    got, ws = sorted_keys_from_the_library(x)
    assert L.lapsum_describe(rows, n).path == L.PATH_BLOCK
    assert_rows_bit_exact(got, x)


@pytest.mark.parametrize("rows,n", [
    # fewer rows than SMs: one thread per pair up to 2048 keys (2 keys per thread), then 4, 8, 16 keys per thread
    (3, 129), (3, 1000), (40, 2048), (40, 4096), (40, 5000), (40, 8192), (40, 16384), (40, 12001),
    # more rows than SMs: 64 / 128 / 512 / 1024 threads, 4 or 8 (16 for the longest rows) keys per thread
    (300, 200), (300, 256), (300, 700), (150, 513), (200, 2048), (200, 3000), (150, 8192), (150, 16384), (150, 9000),
])
def test_block_kernel_sorted_keys(rows, n):
    x = rows_with_ties(rows, n, 20 + n + rows)
    got, ws = sorted_keys_from_the_library(x)
    assert_rows_bit_exact(got, x)


@pytest.mark.parametrize("rows,n", [
    (2, 4096), (2, 2049 * 2 - 1), (30, 4096),      # four blocks per row
    (2, 8192), (2, 16384), (9, 16384), (5, 9001),  # eight blocks per row
    (20, 8192), (20, 16384), (25, 16000),          # rows > 18: four blocks per row, 2 and 4 keys per thread
])
def test_cluster_kernel_sorted_keys(rows, n):
    x = rows_with_ties(rows, n, 30 + n + rows)
    got, ws = sorted_keys_from_the_library(x)
    assert_rows_bit_exact(got, x)


@pytest.mark.parametrize("n", [16385, 8192 * 3 + 1, 100003, 1 << 20, 10_000_000])
def test_keys_only_radix_chain_sorted_keys(n):
    # what lapsum_forward's full-sort chain runs by default: no payload
    x = rows_with_ties(1, n, 40 + n)
    got, ws = sorted_keys_from_the_library(x, L.default_params(force_path=L.PATH_FULLSORT))
    assert ws.params.sort_payload == 0
    assert_rows_bit_exact(got, x)


def test_keys_only_radix_chain_on_a_bracket_workspace_and_a_batch():
    # the default dispatch of long rows (bracket path) keeps the same chain as its fallback; rows > 1 run one by one
    x = rows_with_ties(3, 70001, 77)
    got, ws = sorted_keys_from_the_library(x)
    assert L.lapsum_describe(3, 70001).path == L.PATH_BRACKET
    assert_rows_bit_exact(got, x)


def test_index_payload_needs_a_payload_workspace():
    x = rows_with_ties(1, 20000, 5)
    ws = L.Workspace(1, 20000, L.default_params(force_path=L.PATH_FULLSORT))
    out = torch.empty((1, 20000), device="cuda")
    idx = torch.empty((1, 20000), device="cuda", dtype=torch.int32)
    with pytest.raises(L.LapsumError) as e:
        L.lapsum_debug_sort_pairs(to_dev(x), out, idx, ws)
    assert e.value.code == -8
