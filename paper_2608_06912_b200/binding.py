"""Thin ctypes binding of the C ABI declared in include/lapsum.h.

Argument marshalling only: every step of the solver runs in the CUDA kernels
of liblapsum_b200.so.  PyTorch supplies device memory and streams.  There is
no CPU fallback: if the library is missing or no CUDA device is present the
calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

PATH_AUTO, PATH_BLOCK, PATH_FULLSORT, PATH_BRACKET = 0, 1, 2, 3
PATH_NAMES = {PATH_AUTO: "auto", PATH_BLOCK: "block", PATH_FULLSORT: "fullsort", PATH_BRACKET: "bracket"}

IO_F32, IO_F16, IO_BF16 = 0, 1, 2
IO_TORCH = {IO_F32: torch.float32, IO_F16: torch.float16, IO_BF16: torch.bfloat16}
IO_NAMES = {IO_F32: "f32", IO_F16: "f16", IO_BF16: "bf16"}

ST_FALLBACK = 0x1
ST_BAND_OVERFLOW = 0x2
ST_ROOT_LEFT = 0x4
ST_ROOT_RIGHT = 0x8
ST_LOOKBACK_TIMEOUT = 0x10
ST_NO_CROSSING = 0x20
ST_WIDENED = 0x40
ST_BAD_BUDGET = 0x80
ST_BAD_ALPHA = 0x100
ST_BOUNDS = 0x200

EXPORTS = (
    "lapsum_default_params", "lapsum_workspace_bytes", "lapsum_workspace_init", "lapsum_workspace_release",
    "lapsum_forward", "lapsum_backward", "lapsum_status", "lapsum_debug_sort_pairs", "lapsum_debug_bracket",
    "lapsum_forward_with_bracket", "lapsum_launch_count", "lapsum_error_string", "lapsum_last_cuda_error",
    "lapsum_profile_enable", "lapsum_profile_read", "lapsum_profile_disable", "lapsum_kernel_name",
    "lapsum_backward_static", "lapsum_backward_scalars", "lapsum_forward_backward_host", "lapsum_describe",
    "lapsum_forward_row_budgets", "lapsum_debug_lookback_timeout", "lapsum_forward_rows", "lapsum_backward_rows",
    "lapsum_forward_io", "lapsum_backward_io",
    "lapsum_shard_workspace_bytes", "lapsum_shard_workspace_init", "lapsum_shard_describe", "lapsum_shard_sample",
    "lapsum_shard_stream", "lapsum_shard_solve", "lapsum_shard_mask", "lapsum_shard_vjp_partial", "lapsum_shard_vjp_apply",
)

KERNELS = ("row_block_forward", "row_block_backward", "rs_histogram", "rs_onesweep", "tile_aggregate", "solve_global",
           "cdf_map", "vjp_reduce", "vjp_map", "sample_gather", "stream_band", "misc")


class LapsumError(RuntimeError):
    def __init__(self, code: int, what: str):
        msg = lib().lapsum_error_string(code).decode()
        if code == -6:
            msg += f" (cuda error {lib().lapsum_last_cuda_error()})"
        super().__init__(f"{what}: {msg} [{code}]")
        self.code = code


class Params(C.Structure):
    _fields_ = [
        ("z", C.c_double), ("bracket_min_n", C.c_int64), ("band_capacity", C.c_int64), ("force_path", C.c_int32),
        ("sort_payload", C.c_int32), ("block_max_n", C.c_int32), ("full_sorts", C.c_int32), ("max_widenings", C.c_int32), ("io_dtype", C.c_int32),
    ]


class Plan(C.Structure):
    _fields_ = [
        ("path", C.c_int32), ("reserved", C.c_int32), ("K", C.c_int64), ("stride", C.c_int64),
        ("band_capacity", C.c_int64), ("j", C.c_int64), ("l", C.c_int64), ("workspace_bytes", C.c_size_t),
    ]


class ShardLayout(C.Structure):
    _fields_ = [
        ("K", C.c_int64), ("band_capacity", C.c_int64), ("off_sample_keys", C.c_size_t), ("off_band_count", C.c_size_t),
        ("off_n_R", C.c_size_t), ("off_tails", C.c_size_t), ("off_bucket_counts", C.c_size_t),
        ("off_bucket_sums", C.c_size_t), ("off_band_keys", C.c_size_t), ("off_vjp_sums", C.c_size_t),
    ]


class Stats(C.Structure):
    _fields_ = [
        ("status_bits", C.c_uint32), ("path", C.c_int32), ("forwards", C.c_int64), ("fallbacks", C.c_int64),
        ("widenings", C.c_int64), ("lookback_timeouts", C.c_int64), ("K", C.c_int64), ("j", C.c_int64), ("l", C.c_int64),
        ("a_L", C.c_float), ("a_R", C.c_float), ("n_L", C.c_int64), ("n_M", C.c_int64), ("n_R", C.c_int64),
        ("S_L", C.c_double), ("S_R", C.c_double), ("S_f", C.c_double), ("S_vf", C.c_double),
    ]


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Load (building first if the sources are newer) the CUDA library.  Raises if it cannot be had."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.stale():
            path = _build.build()
        L = C.CDLL(path)
        vp, i64, dbl = C.c_void_p, C.c_int64, C.c_double
        L.lapsum_default_params.argtypes = [C.POINTER(Params)]
        L.lapsum_default_params.restype = None
        L.lapsum_workspace_bytes.argtypes = [i64, i64, C.POINTER(Params), C.POINTER(C.c_size_t)]
        L.lapsum_workspace_init.argtypes = [vp, C.c_size_t, i64, i64, C.POINTER(Params), C.c_uint64, vp]
        L.lapsum_workspace_release.argtypes = [vp]
        L.lapsum_forward.argtypes = [vp, i64, i64, dbl, dbl, vp, vp, vp, vp]
        L.lapsum_backward.argtypes = [vp, vp, vp, dbl, dbl, vp, vp, vp]
        L.lapsum_status.argtypes = [vp, vp, C.POINTER(Stats)]
        L.lapsum_backward_static.argtypes = [vp, vp, vp, i64, i64, dbl, vp, vp]
        L.lapsum_backward_scalars.argtypes = [vp, vp, vp, dbl, dbl, vp, vp, vp, vp, vp]
        L.lapsum_forward_backward_host.argtypes = [vp, vp, i64, i64, dbl, dbl, vp, vp, vp, vp, vp, vp]
        L.lapsum_describe.argtypes = [i64, i64, dbl, C.POINTER(Params), C.POINTER(Plan)]
        L.lapsum_forward_row_budgets.argtypes = [vp, i64, i64, vp, dbl, vp, vp, vp, vp]
        L.lapsum_forward_rows.argtypes = [vp, i64, i64, vp, vp, dbl, dbl, vp, vp, vp, vp]
        L.lapsum_backward_rows.argtypes = [vp, vp, vp, vp, dbl, vp, vp, vp, vp, vp]
        L.lapsum_forward_io.argtypes = [vp, i64, i64, vp, vp, dbl, dbl, vp, vp, vp, vp]
        L.lapsum_backward_io.argtypes = [vp, vp, vp, vp, dbl, vp, vp, vp, vp, vp]
        L.lapsum_shard_workspace_bytes.argtypes = [i64, C.POINTER(Params), C.POINTER(C.c_size_t)]
        L.lapsum_shard_workspace_init.argtypes = [vp, C.c_size_t, i64, C.POINTER(Params), C.c_uint64, vp]
        L.lapsum_shard_describe.argtypes = [vp, C.POINTER(ShardLayout)]
        L.lapsum_shard_sample.argtypes = [vp, i64, i64, i64, dbl, vp, vp]
        L.lapsum_shard_stream.argtypes = [vp, i64, i64, dbl, dbl, vp, vp]
        L.lapsum_shard_solve.argtypes = [i64, dbl, dbl, vp, vp, vp]
        L.lapsum_shard_mask.argtypes = [vp, i64, i64, dbl, vp, vp, vp]
        L.lapsum_shard_vjp_partial.argtypes = [vp, vp, i64, i64, vp, dbl, vp, vp]
        L.lapsum_shard_vjp_apply.argtypes = [vp, vp, i64, i64, vp, dbl, vp, vp, vp, vp, vp]
        L.lapsum_debug_sort_pairs.argtypes = [vp, i64, i64, vp, vp, vp, vp]
        L.lapsum_debug_lookback_timeout.argtypes = [vp, i64, C.c_int, vp, vp]
        L.lapsum_debug_bracket.argtypes = [vp, i64, dbl, dbl, vp, vp, C.c_int, C.c_float, C.c_float, vp, vp]
        L.lapsum_forward_with_bracket.argtypes = [vp, i64, dbl, dbl, C.c_float, C.c_float, vp, vp, vp, vp]
        L.lapsum_launch_count.argtypes = []
        L.lapsum_launch_count.restype = i64
        L.lapsum_error_string.argtypes = [C.c_int]
        L.lapsum_error_string.restype = C.c_char_p
        L.lapsum_last_cuda_error.argtypes = []
        L.lapsum_profile_enable.argtypes = [vp, C.c_uint32, C.c_int]
        L.lapsum_profile_read.argtypes = [vp, vp, C.c_int, C.POINTER(C.c_int64), C.POINTER(C.c_double)]
        L.lapsum_profile_disable.argtypes = [vp]
        L.lapsum_kernel_name.argtypes = [C.c_int]
        L.lapsum_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def default_params(**overrides) -> Params:
    p = Params()
    lib().lapsum_default_params(C.byref(p))
    for key, val in overrides.items():
        if not hasattr(p, key):
            raise AttributeError(key)
        setattr(p, key, val)
    return p


def _check(rc: int, what: str):
    if rc != 0:
        raise LapsumError(rc, what)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _dev_f32(t: torch.Tensor, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous float32 CUDA tensor")
    return t


def lapsum_describe(rows: int, n: int, k: float = 0.0, params: Optional[Params] = None) -> Plan:
    """Host-only: the path, sample size, stride, band capacity, ranks and workspace size for rows x n problems."""
    out = Plan()
    _check(lib().lapsum_describe(rows, n, float(k), C.byref(params) if params is not None else None, C.byref(out)),
           "lapsum_describe")
    return out


def lapsum_workspace_bytes(rows: int, n: int, params: Optional[Params] = None) -> int:
    out = C.c_size_t()
    _check(lib().lapsum_workspace_bytes(rows, n, C.byref(params) if params is not None else None, C.byref(out)),
           "lapsum_workspace_bytes")
    return out.value


def lapsum_launch_count() -> int:
    return lib().lapsum_launch_count()


@dataclass
class StatsView:
    status_bits: int
    path: int
    forwards: int
    fallbacks: int
    widenings: int
    lookback_timeouts: int
    K: int
    j: int
    l: int
    a_L: float
    a_R: float
    n_L: int
    n_M: int
    n_R: int
    S_L: float
    S_R: float
    S_f: float
    S_vf: float


class Workspace:
    """Caller-owned scratch for rows x n problems (lapsum_workspace_bytes / _init / _release)."""

    def __init__(self, rows: int, n: int, params: Optional[Params] = None, seed: int = 0,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("the LapSum library needs a CUDA device; there is no CPU path")
        self.rows, self.n = int(rows), int(n)
        self.params = params if params is not None else default_params()
        self.seed = int(seed)
        self.bytes = lapsum_workspace_bytes(self.rows, self.n, self.params)
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.buf = torch.empty(self.bytes + 256, dtype=torch.uint8, device=dev)
        base = self.buf.data_ptr()
        self.ptr = (base + 255) // 256 * 256
        _check(lib().lapsum_workspace_init(self.ptr, self.bytes, self.rows, self.n, C.byref(self.params),
                                           self.seed, _stream_ptr(stream)), "lapsum_workspace_init")
        self._live = True

    def release(self):
        if getattr(self, "_live", False):
            lib().lapsum_workspace_release(self.ptr)
            self._live = False

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> StatsView:
        s = Stats()
        _check(lib().lapsum_status(self.ptr, _stream_ptr(stream), C.byref(s)), "lapsum_status")
        return StatsView(*[getattr(s, f[0]) for f in Stats._fields_])


def lapsum_profile_enable(ws: "Workspace", kernels=None, max_records: int = 4096) -> None:
    """Bracket launches of the named kernels (default: all) with CUDA events."""
    mask = 0
    for name in (kernels if kernels is not None else KERNELS):
        mask |= 1 << KERNELS.index(name)
    _check(lib().lapsum_profile_enable(ws.ptr, mask, int(max_records)), "lapsum_profile_enable")


def lapsum_profile_read(ws: "Workspace", stream: Optional[torch.cuda.Stream] = None) -> dict:
    """{kernel name: (launches, total ms)} for every kernel with recorded launches."""
    out = {}
    for kid, name in enumerate(KERNELS):
        n, ms = C.c_int64(), C.c_double()
        _check(lib().lapsum_profile_read(ws.ptr, _stream_ptr(stream), kid, C.byref(n), C.byref(ms)),
               "lapsum_profile_read")
        if n.value:
            out[name] = (n.value, ms.value)
    return out


def lapsum_profile_disable(ws: "Workspace") -> None:
    _check(lib().lapsum_profile_disable(ws.ptr), "lapsum_profile_disable")


def lapsum_forward(r: torch.Tensor, k: float, alpha: float, p: torch.Tensor, b: torch.Tensor, ws: Workspace,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
    """p, b <- forward(r) through the C ABI; r, p: rows x n float32, b: rows float32 (all on the GPU)."""
    _dev_f32(r, "r"); _dev_f32(p, "p"); _dev_f32(b, "b")
    rows, n = (1, r.numel()) if r.dim() == 1 else r.shape
    if p.numel() != r.numel() or b.numel() != rows:
        raise ValueError("p must match r and b must hold one value per row")
    _check(lib().lapsum_forward(r.data_ptr(), rows, n, float(k), float(alpha), p.data_ptr(), b.data_ptr(), ws.ptr,
                                _stream_ptr(stream)), "lapsum_forward")


def lapsum_forward_row_budgets(r: torch.Tensor, k_rows: torch.Tensor, alpha: float, p: torch.Tensor, b: torch.Tensor,
                               ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    """lapsum_forward with one budget per row: k_rows is a float64 tensor of rows values on the GPU (block path only)."""
    _dev_f32(r, "r"); _dev_f32(p, "p"); _dev_f32(b, "b")
    if not (k_rows.is_cuda and k_rows.dtype == torch.float64 and k_rows.is_contiguous()):
        raise TypeError("k_rows must be a contiguous float64 CUDA tensor")
    rows, n = (1, r.numel()) if r.dim() == 1 else r.shape
    if p.numel() != r.numel() or b.numel() != rows or k_rows.numel() != rows:
        raise ValueError("p must match r; b and k_rows must hold one value per row")
    _check(lib().lapsum_forward_row_budgets(r.data_ptr(), rows, n, k_rows.data_ptr(), float(alpha), p.data_ptr(),
                                            b.data_ptr(), ws.ptr, _stream_ptr(stream)), "lapsum_forward_row_budgets")


def _dev_f64_rows(t: Optional[torch.Tensor], rows: int, name: str) -> Optional[int]:
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == torch.float64 and t.is_contiguous() and t.numel() == rows):
        raise TypeError(f"{name} must be a contiguous float64 CUDA tensor with one value per row")
    return t.data_ptr()


def lapsum_forward_rows(r: torch.Tensor, k_rows: Optional[torch.Tensor], alpha_rows: Optional[torch.Tensor], k: float,
                        alpha: float, p: torch.Tensor, b: torch.Tensor, ws: Workspace,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """lapsum_forward with one budget and / or one temperature per row (float64 CUDA tensors of rows values, or None
    for the scalar k / alpha)."""
    _dev_f32(r, "r"); _dev_f32(p, "p"); _dev_f32(b, "b")
    rows, n = (1, r.numel()) if r.dim() == 1 else r.shape
    if p.numel() != r.numel() or b.numel() != rows:
        raise ValueError("p must match r and b must hold one value per row")
    _check(lib().lapsum_forward_rows(r.data_ptr(), rows, n, _dev_f64_rows(k_rows, rows, "k_rows"),
                                     _dev_f64_rows(alpha_rows, rows, "alpha_rows"), float(k), float(alpha), p.data_ptr(),
                                     b.data_ptr(), ws.ptr, _stream_ptr(stream)), "lapsum_forward_rows")


def lapsum_backward_rows(v: torch.Tensor, r: torch.Tensor, b: torch.Tensor, alpha_rows: Optional[torch.Tensor],
                         alpha: float, grad_r: torch.Tensor, grad_k: Optional[torch.Tensor],
                         grad_alpha: Optional[torch.Tensor], ws: Workspace,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
    """lapsum_backward_scalars with one temperature per row (float64 CUDA tensor of rows values, or None)."""
    _dev_f32(v, "v"); _dev_f32(r, "r"); _dev_f32(b, "b"); _dev_f32(grad_r, "grad_r")
    for name, t in (("grad_k", grad_k), ("grad_alpha", grad_alpha)):
        if t is not None:
            _dev_f32(t, name)
            if t.numel() != ws.rows:
                raise ValueError(f"{name} must hold one value per row")
    if v.numel() != r.numel() or grad_r.numel() != r.numel() or r.numel() != ws.rows * ws.n or b.numel() != ws.rows:
        raise ValueError("shapes must match the workspace")
    _check(lib().lapsum_backward_rows(v.data_ptr(), r.data_ptr(), b.data_ptr(), _dev_f64_rows(alpha_rows, ws.rows, "alpha_rows"),
                                      float(alpha), grad_r.data_ptr(), grad_k.data_ptr() if grad_k is not None else None,
                                      grad_alpha.data_ptr() if grad_alpha is not None else None, ws.ptr,
                                      _stream_ptr(stream)), "lapsum_backward_rows")


def _dev_io(t: torch.Tensor, ws: "Workspace", name: str) -> torch.Tensor:
    want = IO_TORCH[ws.params.io_dtype]
    if not (t.is_cuda and t.dtype == want and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous {want} CUDA tensor (the workspace's io_dtype)")
    return t


def lapsum_forward_io(r: torch.Tensor, k_rows: Optional[torch.Tensor], alpha_rows: Optional[torch.Tensor], k: float,
                      alpha: float, p: torch.Tensor, b: torch.Tensor, ws: Workspace,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
    """Forward for any storage type: r and p are tensors of the workspace's io_dtype (float32, float16 or bfloat16),
    b float32; k_rows / alpha_rows as in lapsum_forward_rows (None: the scalars k / alpha serve every row)."""
    _dev_io(r, ws, "r"); _dev_io(p, ws, "p"); _dev_f32(b, "b")
    rows, n = (1, r.numel()) if r.dim() == 1 else r.shape
    if p.numel() != r.numel() or b.numel() != rows:
        raise ValueError("p must match r and b must hold one value per row")
    _check(lib().lapsum_forward_io(r.data_ptr(), rows, n, _dev_f64_rows(k_rows, rows, "k_rows"),
                                   _dev_f64_rows(alpha_rows, rows, "alpha_rows"), float(k), float(alpha), p.data_ptr(),
                                   b.data_ptr(), ws.ptr, _stream_ptr(stream)), "lapsum_forward_io")


def lapsum_backward_io(v: torch.Tensor, r: torch.Tensor, b: torch.Tensor, alpha_rows: Optional[torch.Tensor], alpha: float,
                       grad_r: torch.Tensor, grad_k: Optional[torch.Tensor], grad_alpha: Optional[torch.Tensor],
                       ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Backward for any storage type: v, r, grad_r are tensors of the workspace's io_dtype, b, grad_k, grad_alpha float32."""
    _dev_io(v, ws, "v"); _dev_io(r, ws, "r"); _dev_io(grad_r, ws, "grad_r"); _dev_f32(b, "b")
    for name, t in (("grad_k", grad_k), ("grad_alpha", grad_alpha)):
        if t is not None:
            _dev_f32(t, name)
            if t.numel() != ws.rows:
                raise ValueError(f"{name} must hold one value per row")
    if v.numel() != r.numel() or grad_r.numel() != r.numel() or r.numel() != ws.rows * ws.n or b.numel() != ws.rows:
        raise ValueError("shapes must match the workspace")
    _check(lib().lapsum_backward_io(v.data_ptr(), r.data_ptr(), b.data_ptr(), _dev_f64_rows(alpha_rows, ws.rows, "alpha_rows"),
                                    float(alpha), grad_r.data_ptr(), grad_k.data_ptr() if grad_k is not None else None,
                                    grad_alpha.data_ptr() if grad_alpha is not None else None, ws.ptr,
                                    _stream_ptr(stream)), "lapsum_backward_io")


def lapsum_backward(v: torch.Tensor, r: torch.Tensor, b: torch.Tensor, k: float, alpha: float, grad_r: torch.Tensor,
                    ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    _dev_f32(v, "v"); _dev_f32(r, "r"); _dev_f32(b, "b"); _dev_f32(grad_r, "grad_r")
    if v.numel() != r.numel() or grad_r.numel() != r.numel() or r.numel() != ws.rows * ws.n or b.numel() != ws.rows:
        raise ValueError("shapes must match the workspace")
    _check(lib().lapsum_backward(v.data_ptr(), r.data_ptr(), b.data_ptr(), float(k), float(alpha), grad_r.data_ptr(),
                                 ws.ptr, _stream_ptr(stream)), "lapsum_backward")


def _host_f32(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous float32 host tensor")
    return t


def lapsum_forward_backward_host(r_host: torch.Tensor, v_host: torch.Tensor, k: float, alpha: float,
                                 p_host: torch.Tensor, grad_host: torch.Tensor, b_host: torch.Tensor,
                                 staging: torch.Tensor, ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    """One forward + backward from host tensors (page-locked for overlap) into host tensors.  `staging` is a
    float32 CUDA tensor of at least 4*rows*n + rows elements.  Results are complete once `stream` has finished."""
    for name, t in (("r_host", r_host), ("v_host", v_host), ("p_host", p_host), ("grad_host", grad_host),
                    ("b_host", b_host)):
        _host_f32(t, name)
    _dev_f32(staging, "staging")
    N = ws.rows * ws.n
    if any(t.numel() != N for t in (r_host, v_host, p_host, grad_host)) or b_host.numel() != ws.rows:
        raise ValueError("shapes must match the workspace")
    if staging.numel() < 4 * N + ws.rows:
        raise ValueError("staging must hold 4*rows*n + rows floats")
    _check(lib().lapsum_forward_backward_host(r_host.data_ptr(), v_host.data_ptr(), ws.rows, ws.n, float(k), float(alpha),
                                              p_host.data_ptr(), grad_host.data_ptr(), b_host.data_ptr(),
                                              staging.data_ptr(), ws.ptr, _stream_ptr(stream)),
           "lapsum_forward_backward_host")


def lapsum_backward_scalars(v: torch.Tensor, r: torch.Tensor, b: torch.Tensor, k: float, alpha: float,
                            grad_r: torch.Tensor, grad_k: Optional[torch.Tensor], grad_alpha: Optional[torch.Tensor],
                            ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    """lapsum_backward plus the per-row gradients of the budget k and of the temperature alpha."""
    _dev_f32(v, "v"); _dev_f32(r, "r"); _dev_f32(b, "b"); _dev_f32(grad_r, "grad_r")
    for name, t in (("grad_k", grad_k), ("grad_alpha", grad_alpha)):
        if t is not None:
            _dev_f32(t, name)
            if t.numel() != ws.rows:
                raise ValueError(f"{name} must hold one value per row")
    if v.numel() != r.numel() or grad_r.numel() != r.numel() or r.numel() != ws.rows * ws.n or b.numel() != ws.rows:
        raise ValueError("shapes must match the workspace")
    _check(lib().lapsum_backward_scalars(v.data_ptr(), r.data_ptr(), b.data_ptr(), float(k), float(alpha),
                                         grad_r.data_ptr(), grad_k.data_ptr() if grad_k is not None else None,
                                         grad_alpha.data_ptr() if grad_alpha is not None else None, ws.ptr,
                                         _stream_ptr(stream)), "lapsum_backward_scalars")


STATIC_MAX_ROWS = 65536


def lapsum_backward_static(v: torch.Tensor, r: torch.Tensor, b: torch.Tensor, alpha: float, grad_r: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """Backward for callers that may not allocate: no workspace, scratch lives inside the library.

    Same result as lapsum_backward on a workspace of a long-row path.  rows <= 65536.  The first call on a
    device resolves the scratch address (do it before any stream capture); calls that overlap on the GPU
    race on the shared scratch, so keep them on one stream or order them.
    """
    _dev_f32(v, "v"); _dev_f32(r, "r"); _dev_f32(b, "b"); _dev_f32(grad_r, "grad_r")
    rows, n = (1, r.numel()) if r.dim() == 1 else r.shape
    if v.numel() != r.numel() or grad_r.numel() != r.numel() or b.numel() != rows:
        raise ValueError("v and grad_r must match r, b must hold one value per row")
    _check(lib().lapsum_backward_static(v.data_ptr(), r.data_ptr(), b.data_ptr(), rows, n, float(alpha),
                                        grad_r.data_ptr(), _stream_ptr(stream)), "lapsum_backward_static")


def lapsum_forward_with_bracket(r: torch.Tensor, k: float, alpha: float, a_L: float, a_R: float, p: torch.Tensor,
                                b: torch.Tensor, ws: Workspace, stream: Optional[torch.cuda.Stream] = None) -> None:
    _dev_f32(r, "r"); _dev_f32(p, "p"); _dev_f32(b, "b")
    _check(lib().lapsum_forward_with_bracket(r.data_ptr(), r.numel(), float(k), float(alpha), a_L, a_R, p.data_ptr(),
                                             b.data_ptr(), ws.ptr, _stream_ptr(stream)), "lapsum_forward_with_bracket")


def lapsum_debug_sort_pairs(keys: torch.Tensor, keys_out: torch.Tensor, idx_out: Optional[torch.Tensor], ws: Workspace,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """Sorted rows (and, with idx_out, the original indices) from the library's sort kernels; idx_out = None runs
    the very kernels the forward sorts with (see include/lapsum.h)."""
    _dev_f32(keys, "keys"); _dev_f32(keys_out, "keys_out")
    if idx_out is not None and not (idx_out.is_cuda and idx_out.dtype == torch.int32 and idx_out.is_contiguous()):
        raise TypeError("idx_out must be a contiguous int32 CUDA tensor (bit pattern of uint32)")
    rows, n = (1, keys.numel()) if keys.dim() == 1 else keys.shape
    _check(lib().lapsum_debug_sort_pairs(keys.data_ptr(), rows, n, keys_out.data_ptr(),
                                         idx_out.data_ptr() if idx_out is not None else None, ws.ptr,
                                         _stream_ptr(stream)), "lapsum_debug_sort_pairs")


def lapsum_debug_lookback_timeout(keys: torch.Tensor, spin_limit: int, ws: Workspace,
                                  stream: Optional[torch.cuda.Stream] = None) -> None:
    """Run one radix pass whose first tile never publishes its counts, with `spin_limit` polls as the wait's bound."""
    _dev_f32(keys, "keys")
    _check(lib().lapsum_debug_lookback_timeout(keys.data_ptr(), keys.numel(), int(spin_limit), ws.ptr,
                                               _stream_ptr(stream)), "lapsum_debug_lookback_timeout")


def lapsum_debug_bracket(r: torch.Tensor, k: float, alpha: float, ws: Workspace, override=None,
                         y_out: Optional[torch.Tensor] = None, band_out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
    _dev_f32(r, "r")
    use = 0 if override is None else 1
    a_L, a_R = (0.0, 0.0) if override is None else override
    _check(lib().lapsum_debug_bracket(r.data_ptr(), r.numel(), float(k), float(alpha), ws.ptr, _stream_ptr(stream),
                                      use, a_L, a_R, y_out.data_ptr() if y_out is not None else None,
                                      band_out.data_ptr() if band_out is not None else None), "lapsum_debug_bracket")


def band_capacity(ws: Workspace) -> int:
    """Elements the middle-band buffer of a bracket-path workspace holds (asked of the library: lapsum_describe)."""
    return int(lapsum_describe(ws.rows, ws.n, 0.0, ws.params).band_capacity)


class ShardWorkspace:
    """Workspace of ONE shard of a row that is spread over several GPUs (lapsum_shard_workspace_bytes / _init), with
    tensor views of the buffers the caller's collectives merge in place (lapsum_shard_describe)."""

    def __init__(self, n_total: int, params: Optional[Params] = None, seed: int = 0,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("the LapSum library needs a CUDA device; there is no CPU path")
        self.rows, self.n = 1, int(n_total)
        self.params = params if params is not None else default_params()
        self.seed = int(seed)
        out = C.c_size_t()
        _check(lib().lapsum_shard_workspace_bytes(self.n, C.byref(self.params), C.byref(out)), "lapsum_shard_workspace_bytes")
        self.bytes = out.value
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.buf = torch.empty(self.bytes + 256, dtype=torch.uint8, device=dev)
        self.ptr = (self.buf.data_ptr() + 255) // 256 * 256
        _check(lib().lapsum_shard_workspace_init(self.ptr, self.bytes, self.n, C.byref(self.params), self.seed,
                                                 _stream_ptr(stream)), "lapsum_shard_workspace_init")
        self._live = True
        lay = ShardLayout()
        _check(lib().lapsum_shard_describe(self.ptr, C.byref(lay)), "lapsum_shard_describe")
        self.K, self.band_capacity = int(lay.K), int(lay.band_capacity)
        base = self.ptr - self.buf.data_ptr()

        def view(off, count, dtype, esz):
            return self.buf[base + off: base + off + count * esz].view(dtype)

        self.sample_keys = view(lay.off_sample_keys, self.K, torch.int32, 4)
        self.band_count = view(lay.off_band_count, 1, torch.int64, 8)
        self.n_R = view(lay.off_n_R, 1, torch.int64, 8)
        self.tails = view(lay.off_tails, 2, torch.float64, 8)
        self.bucket_counts = view(lay.off_bucket_counts, 1024, torch.int32, 4)
        self.bucket_sums = view(lay.off_bucket_sums, 2048, torch.int64, 8)
        self.band_keys = view(lay.off_band_keys, self.band_capacity, torch.int32, 4)
        self.vjp_sums = view(lay.off_vjp_sums, 4, torch.float64, 8)

    def release(self):
        if getattr(self, "_live", False):
            lib().lapsum_workspace_release(self.ptr)
            self._live = False

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> StatsView:
        s = Stats()
        _check(lib().lapsum_status(self.ptr, _stream_ptr(stream), C.byref(s)), "lapsum_status")
        return StatsView(*[getattr(s, f[0]) for f in Stats._fields_])


class GpuShard:
    """One contiguous shard of a row on this GPU: the per-shard steps of the sharded solver (dist.forward_sharded /
    dist.backward_sharded drive them and merge what they leave in the workspace's exchange buffers)."""

    def __init__(self, r_shard: torch.Tensor, begin: int, n_total: int, params: Optional[Params] = None, seed: int = 0,
                 stream: Optional[torch.cuda.Stream] = None):
        _dev_f32(r_shard, "r_shard")
        self.r, self.begin, self.n_total, self.len = r_shard, int(begin), int(n_total), r_shard.numel()
        self.ws = ShardWorkspace(n_total, params, seed, r_shard.device, stream)
        self.stream = stream
        self.p = torch.empty_like(r_shard)
        self.b = torch.empty(1, device=r_shard.device)
        self.grad = None
        self.grad_k = torch.empty(1, device=r_shard.device)
        self.grad_alpha = torch.empty(1, device=r_shard.device)
        w = self.ws
        self.band_capacity = w.band_capacity
        self.sample_keys, self.band_count, self.n_R, self.tails = w.sample_keys, w.band_count, w.n_R, w.tails
        self.bucket_counts, self.bucket_sums, self.band_keys, self.vjp_sums = (w.bucket_counts, w.bucket_sums, w.band_keys,
                                                                               w.vjp_sums)

    def _st(self):
        return _stream_ptr(self.stream)

    def sample(self, alpha: float) -> None:
        _check(lib().lapsum_shard_sample(self.r.data_ptr(), self.begin, self.len, self.n_total, float(alpha), self.ws.ptr,
                                         self._st()), "lapsum_shard_sample")

    def stream_pass(self, k: float, alpha: float) -> None:
        _check(lib().lapsum_shard_stream(self.r.data_ptr(), self.len, self.n_total, float(k), float(alpha), self.ws.ptr,
                                         self._st()), "lapsum_shard_stream")

    def solve(self, k: float, alpha: float) -> None:
        _check(lib().lapsum_shard_solve(self.n_total, float(k), float(alpha), self.b.data_ptr(), self.ws.ptr, self._st()),
               "lapsum_shard_solve")

    def mask(self, alpha: float) -> None:
        _check(lib().lapsum_shard_mask(self.r.data_ptr(), self.len, self.n_total, float(alpha), self.p.data_ptr(), self.ws.ptr,
                                       self._st()), "lapsum_shard_mask")

    def vjp_partial(self, v_shard: torch.Tensor, alpha: float) -> None:
        _dev_f32(v_shard, "v_shard")
        _check(lib().lapsum_shard_vjp_partial(v_shard.data_ptr(), self.r.data_ptr(), self.len, self.n_total, self.b.data_ptr(),
                                              float(alpha), self.ws.ptr, self._st()), "lapsum_shard_vjp_partial")

    def vjp_apply(self, v_shard: torch.Tensor, alpha: float) -> None:
        if self.grad is None:
            self.grad = torch.empty_like(self.r)
        _check(lib().lapsum_shard_vjp_apply(v_shard.data_ptr(), self.r.data_ptr(), self.len, self.n_total, self.b.data_ptr(),
                                            float(alpha), self.grad.data_ptr(), self.grad_k.data_ptr(),
                                            self.grad_alpha.data_ptr(), self.ws.ptr, self._st()), "lapsum_shard_vjp_apply")

    def whole_row_forward(self, r_full: torch.Tensor, k: float, alpha: float) -> None:
        """The rare way out when the bracket's certificate failed: the whole row on this GPU, ordinary forward."""
        ws = Workspace(1, self.n_total, self.ws.params, self.ws.seed, r_full.device, self.stream)
        p_full = torch.empty_like(r_full)
        lapsum_forward(r_full, k, alpha, p_full, self.b, ws, self.stream)
        self.p.copy_(p_full.view(-1)[self.begin:self.begin + self.len])
        ws.release()
