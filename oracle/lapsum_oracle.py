"""ctypes front end of the CPU oracle (oracle/lapsum_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module.
The shared object is compiled on first use with gcc (fp64, single thread,
no fused contractions).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lapsum_oracle.c")
_LIB = os.path.join(_HERE, "liblapsum_oracle.so")

ROOT_LEFT = 1
ROOT_RIGHT = 2


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _SolveInfo(C.Structure):
    _fields_ = [
        ("b", C.c_double), ("jstar", C.c_int64), ("c", C.c_double), ("A", C.c_double), ("Bs", C.c_double),
        ("lo", C.c_double), ("hi", C.c_double), ("F_aL", C.c_double), ("F_aR", C.c_double), ("status", C.c_int),
    ]


class _BracketInfo(C.Structure):
    _fields_ = [
        ("K", C.c_int64), ("j", C.c_int64), ("l", C.c_int64), ("a_L", C.c_float), ("a_R", C.c_float),
        ("n_L", C.c_int64), ("n_M", C.c_int64), ("n_R", C.c_int64), ("S_L", C.c_double), ("S_R", C.c_double),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, dp, ip = C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int64)
        L.oracle_sort_pairs.argtypes = [fp, C.c_int64, fp, C.POINTER(C.c_uint32)]
        L.oracle_lap_sum.argtypes = [fp, C.c_int64, C.c_double, C.c_double]
        L.oracle_lap_sum.restype = C.c_double
        L.oracle_bisect.argtypes = [fp, C.c_int64, C.c_double, C.c_double, dp]
        L.oracle_solve_sorted.argtypes = [dp, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_double,
                                          C.c_double, C.c_double, C.c_int64, dp, C.POINTER(_SolveInfo)]
        L.oracle_forward.argtypes = [fp, C.c_int64, C.c_int64, C.c_double, C.c_double, dp, dp, ip, dp]
        L.oracle_backward.argtypes = [fp, fp, dp, C.c_int64, C.c_int64, C.c_double, dp]
        L.oracle_backward_scalars.argtypes = [fp, fp, dp, C.c_int64, C.c_int64, C.c_double, dp, dp]
        L.oracle_sample_count.argtypes = [C.c_int64]
        L.oracle_sample_count.restype = C.c_int64
        L.oracle_bracket_indices.argtypes = [C.c_int64, C.c_double, C.c_double, ip, ip, ip]
        L.oracle_bracket_indices.restype = None
        L.oracle_noise.argtypes = [C.c_uint64, C.c_int64]
        L.oracle_noise.restype = C.c_float
        L.oracle_sample_index.argtypes = [C.c_uint64, C.c_int64, C.c_int64, C.c_int64]
        L.oracle_sample_index.restype = C.c_int64
        L.oracle_noise_table.argtypes = [C.c_uint64, C.c_int64, fp]
        L.oracle_noise_table.restype = None
        L.oracle_sample_indices.argtypes = [C.c_uint64, C.c_int64, C.c_int64, ip]
        L.oracle_sample_indices.restype = None
        L.oracle_widen.argtypes = [C.c_float, C.c_float, C.c_double, C.c_int, C.POINTER(C.c_float),
                                   C.POINTER(C.c_float)]
        L.oracle_forward_validated.argtypes = [fp, C.c_int64, C.c_double, C.c_double, C.c_float, C.c_float, C.c_int,
                                               dp, dp, ip, fp, ip, dp]
        L.oracle_bracket.argtypes = [fp, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_uint64, fp,
                                     C.POINTER(_BracketInfo)]
        L.oracle_forward_bracketed.argtypes = [fp, C.c_int64, C.c_double, C.c_double, C.c_float, C.c_float,
                                               dp, dp, C.POINTER(C.c_int), ip, dp, fp, C.c_int64]
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float)) if a is not None else None


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double)) if a is not None else None


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int64)) if a is not None else None


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"{what}: oracle returned {rc}")


def sort_pairs(r):
    """Ascending (key, original index) of one row under the total order on fp32 bit patterns."""
    r = _f32(r).ravel()
    keys = np.empty_like(r)
    idx = np.empty(r.shape[0], dtype=np.uint32)
    _check(lib().oracle_sort_pairs(_fp(r), r.shape[0], _fp(keys), idx.ctypes.data_as(C.POINTER(C.c_uint32))),
           "sort_pairs")
    return keys, idx


def lap_sum(r, b: float, t: float) -> float:
    r = _f32(r).ravel()
    return lib().oracle_lap_sum(_fp(r), r.shape[0], float(b), float(t))


def bisect(r, k: float, alpha: float) -> float:
    r = _f32(r).ravel()
    out = C.c_double()
    _check(lib().oracle_bisect(_fp(r), r.shape[0], float(k), float(alpha), C.byref(out)), "bisect")
    return out.value


@dataclass
class Forward:
    p: np.ndarray | None
    b: np.ndarray
    jstar: np.ndarray
    node_F: np.ndarray | None


def forward(r, k: float, alpha: float, want_p: bool = True, want_nodes: bool = False) -> Forward:
    r = _f32(r)
    if r.ndim == 1:
        r = r.reshape(1, -1)
    rows, n = r.shape
    p = np.empty((rows, n), dtype=np.float64) if want_p else None
    b = np.empty(rows, dtype=np.float64)
    js = np.empty(rows, dtype=np.int64)
    nf = np.empty((rows, n + 2), dtype=np.float64) if want_nodes else None
    _check(lib().oracle_forward(_fp(r), rows, n, float(k), float(alpha), _dp(p), _dp(b), _ip(js), _dp(nf)),
           "forward")
    return Forward(p, b, js, nf)


def backward(v, r, b, alpha: float) -> np.ndarray:
    r = _f32(r)
    v = _f32(v)
    if r.ndim == 1:
        r = r.reshape(1, -1)
        v = v.reshape(1, -1)
    rows, n = r.shape
    b = np.ascontiguousarray(np.broadcast_to(np.asarray(b, dtype=np.float64).ravel(), (rows,)))
    g = np.empty((rows, n), dtype=np.float64)
    _check(lib().oracle_backward(_fp(v), _fp(r), _dp(b), rows, n, float(alpha), _dp(g)), "backward")
    return g


def backward_scalars(v, r, b, alpha: float):
    """(grad_k, grad_alpha) per row of L = sum_i v_i p_i."""
    r = _f32(r)
    v = _f32(v)
    if r.ndim == 1:
        r = r.reshape(1, -1)
        v = v.reshape(1, -1)
    rows, n = r.shape
    b = np.ascontiguousarray(np.broadcast_to(np.asarray(b, dtype=np.float64).ravel(), (rows,)))
    gk = np.empty(rows, dtype=np.float64)
    ga = np.empty(rows, dtype=np.float64)
    _check(lib().oracle_backward_scalars(_fp(v), _fp(r), _dp(b), rows, n, float(alpha), _dp(gk), _dp(ga)),
           "backward_scalars")
    return gk, ga


@dataclass
class Solve:
    b: float
    jstar: int
    c: float
    A: float
    Bs: float
    lo: float
    hi: float
    F_aL: float
    F_aR: float
    status: int
    node_F: np.ndarray | None


def solve_sorted(x, k, t, a_L=-np.inf, S_L=0.0, a_R=np.inf, S_R=0.0, n_R=0, want_nodes=False) -> Solve:
    x = np.ascontiguousarray(x, dtype=np.float64).ravel()
    M = x.shape[0]
    nf = np.empty(M + 2, dtype=np.float64) if want_nodes else None
    info = _SolveInfo()
    _check(lib().oracle_solve_sorted(_dp(x), M, float(k), float(t), float(a_L), float(S_L), float(a_R),
                                     float(S_R), int(n_R), _dp(nf), C.byref(info)), "solve_sorted")
    return Solve(info.b, info.jstar, info.c, info.A, info.Bs, info.lo, info.hi, info.F_aL, info.F_aR,
                 info.status, nf)


def sample_count(n: int) -> int:
    return lib().oracle_sample_count(int(n))


def bracket_indices(n: int, k: float, z: float = 5.16):
    K, j, l = C.c_int64(), C.c_int64(), C.c_int64()
    lib().oracle_bracket_indices(int(n), float(k), float(z), C.byref(K), C.byref(j), C.byref(l))
    return K.value, j.value, l.value


def noise_table(seed: int, K: int) -> np.ndarray:
    out = np.empty(int(K), dtype=np.float32)
    lib().oracle_noise_table(int(seed), int(K), _fp(out))
    return out


def sample_indices(seed: int, n: int, K: int) -> np.ndarray:
    out = np.empty(int(K), dtype=np.int64)
    lib().oracle_sample_indices(int(seed), int(n), int(K), _ip(out))
    return out


@dataclass
class Bracket:
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
    y: np.ndarray


def bracket(r, k: float, alpha: float, z: float = 5.16, seed: int = 0) -> Bracket:
    r = _f32(r).ravel()
    n = r.shape[0]
    K = sample_count(n)
    y = np.empty(K, dtype=np.float32)
    info = _BracketInfo()
    _check(lib().oracle_bracket(_fp(r), n, float(k), float(alpha), float(z), int(seed), _fp(y), C.byref(info)),
           "bracket")
    return Bracket(info.K, info.j, info.l, info.a_L, info.a_R, info.n_L, info.n_M, info.n_R, info.S_L,
                   info.S_R, y)


@dataclass
class Bracketed:
    p: np.ndarray | None
    b: float
    status: int
    n_L: int
    n_M: int
    n_R: int
    S_L: float
    S_R: float
    band: np.ndarray | None


@dataclass
class Validated:
    p: np.ndarray | None
    b: float
    widenings: int
    full_sort: bool
    a_L: float  # the last bracket tried
    a_R: float
    n_L: int
    n_M: int
    n_R: int
    S_L: float
    S_R: float


def widen(a_L, a_R, t, status):
    """One-sided doubling of a failed bracket (fp32 ends); None when no finite widened bracket exists."""
    nl, nr = C.c_float(), C.c_float()
    rc = lib().oracle_widen(C.c_float(a_L), C.c_float(a_R), C.c_double(t), int(status), C.byref(nl), C.byref(nr))
    return None if rc else (nl.value, nr.value)


def forward_validated(r, k, alpha, a_L, a_R, max_widen=2, want_p=True) -> Validated:
    """The validated bracket path: solve, widen on a failed certificate, full sort after max_widen."""
    r = _f32(r).ravel()
    n = r.shape[0]
    p = np.empty(n, dtype=np.float64) if want_p else None
    b = C.c_double()
    info = np.zeros(2, dtype=np.int64)
    ends = np.zeros(2, dtype=np.float32)
    counts = np.zeros(3, dtype=np.int64)
    tails = np.zeros(2, dtype=np.float64)
    _check(lib().oracle_forward_validated(_fp(r), n, C.c_double(k), C.c_double(alpha), C.c_float(a_L), C.c_float(a_R),
                                          int(max_widen), _dp(p), C.byref(b), _ip(info), _fp(ends), _ip(counts),
                                          _dp(tails)), "forward_validated")
    return Validated(p, b.value, int(info[0]), bool(info[1]), float(ends[0]), float(ends[1]), int(counts[0]),
                     int(counts[1]), int(counts[2]), float(tails[0]), float(tails[1]))


def forward_bracketed(r, k, alpha, a_L, a_R, want_p=True, want_band=False) -> Bracketed:
    r = _f32(r).ravel()
    n = r.shape[0]
    p = np.empty(n, dtype=np.float64) if want_p else None
    b = C.c_double()
    st = C.c_int()
    counts = np.zeros(3, dtype=np.int64)
    tails = np.zeros(2, dtype=np.float64)
    band = np.empty(n, dtype=np.float32) if want_band else None
    _check(lib().oracle_forward_bracketed(_fp(r), n, float(k), float(alpha), C.c_float(a_L), C.c_float(a_R),
                                          _dp(p), C.byref(b), C.byref(st), _ip(counts), _dp(tails),
                                          _fp(band), n if want_band else 0), "forward_bracketed")
    if band is not None:
        band = band[: counts[1]].copy()
    if st.value != 0:
        p = None
    return Bracketed(p, b.value, st.value, int(counts[0]), int(counts[1]), int(counts[2]), float(tails[0]),
                     float(tails[1]), band)
