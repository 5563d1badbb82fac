"""ctypes front end of the CPU oracle (``omse_oracle.c``).

TEST INFRASTRUCTURE ONLY: the CUDA library never imports this module.  It compiles the
C file with gcc on first use and exposes the oracle's functions on numpy arrays.
Every function's arithmetic lives in the C file; this module only marshals arguments.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "omse_oracle.c")
_LIB = os.path.join(_HERE, "libomse_oracle.so")

STATUS_NONFINITE = 1
STATUS_DEGENERATE = 2


def build(force: bool = False) -> str:
    """Compile the oracle (no fast-math, no contraction) and return the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = C.CDLL(build())
    f32p, f64p = C.POINTER(C.c_float), C.POINTER(C.c_double)
    i32p, i8p, u8p, u32p = C.POINTER(C.c_int32), C.POINTER(C.c_int8), C.POINTER(C.c_uint8), C.POINTER(C.c_uint32)
    lib.omse_oracle_max_threads.restype = C.c_int
    lib.omse_oracle_grid_bounds.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.omse_oracle_sse_at.restype = C.c_double
    lib.omse_oracle_sse_at.argtypes = [f32p, C.c_int64, C.c_float, C.c_int, C.c_int]
    lib.omse_oracle_codes.argtypes = [f32p, C.c_int64, C.c_float, C.c_int, C.c_int, i8p]
    lib.omse_oracle_candidate.restype = C.c_float
    lib.omse_oracle_candidate.argtypes = [C.c_float, C.c_float, C.c_int, C.c_int]
    lib.omse_oracle_phi.argtypes = [f32p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int,
                                    f32p, f64p, i32p, i8p, f64p, u32p]
    lib.omse_oracle_quantize_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float,
                                              C.c_int, i32p, f32p, f64p, i32p, i8p, u32p]
    lib.omse_oracle_activation_scale.argtypes = [f32p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int,
                                                 f32p, f64p, i32p, f64p, u32p]
    lib.omse_oracle_residual_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.POINTER(C.c_int), C.c_int, C.c_int,
                                              C.c_float, C.c_int, C.c_int, C.c_int, f32p, f64p, i32p, i8p, u32p]
    lib.omse_oracle_dual_sse_at.restype = C.c_double
    lib.omse_oracle_dual_sse_at.argtypes = [f32p, C.c_int64, C.c_float, C.c_float, C.c_int, C.c_int, C.c_int]
    lib.omse_oracle_dual_scales.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int, C.c_int, C.c_int, C.c_int,
                                            f32p, f32p]
    lib.omse_oracle_dual.argtypes = [f32p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float,
                                     C.c_float, C.c_int, f32p, f64p, i32p, i8p, i8p, f64p, u32p]
    lib.omse_oracle_dual_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                          C.c_float, C.c_float, i32p, f32p, f64p, i32p, i8p, u32p]
    lib.omse_oracle_layer_mse.restype = C.c_double
    lib.omse_oracle_layer_mse.argtypes = [f32p, C.c_int64, C.c_int64]
    lib.omse_oracle_compression_ratio.restype = C.c_double
    lib.omse_oracle_compression_ratio.argtypes = [C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int),
                                                  C.POINTER(C.c_int), C.c_int]
    lib.omse_oracle_alg1_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int,
                                          C.c_float, C.c_int, C.c_int, C.c_int, f32p, f64p, i32p, i8p, f64p, u32p]
    lib.omse_oracle_offset_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_int, i32p,
                                            f32p, f32p, f64p, i32p, i8p, u32p]
    lib.omse_oracle_alg1_rows_eps.argtypes = [f32p, C.c_int64, C.c_int64, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                              C.c_int, C.c_float, C.c_int, C.c_int, C.c_int, C.c_double, f32p, f64p,
                                              i32p, i8p, f64p, i32p, u32p]
    lib.omse_oracle_solver_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float,
                                            C.c_int, f32p, f64p, i8p, u32p]
    lib.omse_oracle_solver_phi.argtypes = [f32p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int,
                                           f32p, f64p, i8p, i32p, u32p]
    lib.omse_oracle_affine_rows.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_int,
                                            C.c_float, C.c_int, i32p, f32p, f32p, f64p, i32p, i8p, u32p]
    lib.omse_oracle_affine_phi.argtypes = [f32p, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_int, C.c_float, C.c_int,
                                           C.c_int, f32p, f32p, f64p, i32p, i8p, f64p, u32p]
    lib.omse_oracle_pack_int4.argtypes = [i8p, C.c_int64, u8p]
    lib.omse_oracle_unpack_int4.argtypes = [u8p, C.c_int64, C.c_int, i8p]
    _lib = lib
    return lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _c32(v) -> float:
    return float(np.float32(v))


def _f32(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def max_threads() -> int:
    return int(_load().omse_oracle_max_threads())


def grid_bounds(bits: int, is_signed: bool):
    lo, hi = C.c_int(), C.c_int()
    _load().omse_oracle_grid_bounds(bits, int(is_signed), C.byref(lo), C.byref(hi))
    return lo.value, hi.value


def candidate(max_abs: float, hi_frac: float, n_cand: int, c: int) -> float:
    return float(_load().omse_oracle_candidate(_c32(max_abs), _c32(hi_frac), n_cand, c))


def sse_at(x, alpha: float, bits: int, is_signed: bool) -> float:
    x = _f32(x).ravel()
    return float(_load().omse_oracle_sse_at(_p(x, C.c_float), x.size, _c32(alpha), bits, int(is_signed)))


def codes(x, alpha: float, bits: int, is_signed: bool) -> np.ndarray:
    x = _f32(x)
    out = np.empty(x.shape, dtype=np.int8)
    _load().omse_oracle_codes(_p(x, C.c_float), x.size, _c32(alpha), bits, int(is_signed), _p(out, C.c_int8))
    return out


@dataclass
class PhiResult:
    alpha: float
    sse: float
    best_idx: int
    codes: np.ndarray | None
    sse_curve: np.ndarray | None
    status: int


def phi(x, bits=4, is_signed=True, n_cand=256, hi_frac=1.0, refine_iters=3, start_idx=-1,
        want_codes=True, want_curve=False) -> PhiResult:
    """The quantization mapping of Section 3.4 on one segment."""
    x = _f32(x).ravel()
    a, s, i, st = C.c_float(), C.c_double(), C.c_int32(), C.c_uint32(0)
    q = np.empty(x.size, dtype=np.int8) if want_codes else None
    curve = np.empty(n_cand, dtype=np.float64) if want_curve else None
    _load().omse_oracle_phi(_p(x, C.c_float), x.size, bits, int(is_signed), n_cand, _c32(hi_frac),
                            refine_iters, start_idx, C.byref(a), C.byref(s), C.byref(i),
                            _p(q, C.c_int8), _p(curve, C.c_double), C.byref(st))
    return PhiResult(a.value, s.value, i.value, q, curve, st.value)


@dataclass
class RowsResult:
    alpha: np.ndarray      # [S] float32
    sse: np.ndarray        # [S] float64
    best_idx: np.ndarray   # [S] int32
    codes: np.ndarray | None  # [S, K] int8
    status: int


def quantize_rows(w, bits=4, is_signed=True, n_cand=256, hi_frac=1.0, refine_iters=3, start_idx=None,
                  want_codes=True) -> RowsResult:
    """Kernel-wise phi over the rows of a 2-D array [n_kernels, kernel_len] (Section 3.3)."""
    w = _f32(w)
    assert w.ndim == 2
    S, K = w.shape
    alpha = np.empty(S, np.float32)
    sse = np.empty(S, np.float64)
    idx = np.empty(S, np.int32)
    q = np.empty((S, K), np.int8) if want_codes else None
    st = C.c_uint32(0)
    si = None if start_idx is None else np.ascontiguousarray(start_idx, dtype=np.int32)
    _load().omse_oracle_quantize_rows(_p(w, C.c_float), S, K, bits, int(is_signed), n_cand, _c32(hi_frac),
                                      refine_iters, _p(si, C.c_int32), _p(alpha, C.c_float), _p(sse, C.c_double),
                                      _p(idx, C.c_int32), _p(q, C.c_int8), C.byref(st))
    return RowsResult(alpha, sse, idx, q, st.value)


def activation_scale(x, bits=4, is_signed=False, n_cand=2048, hi_frac=1.0, refine_iters=3,
                     want_curve=True) -> PhiResult:
    """Per-tensor phi (Section 3.7) with the candidates spread over the host threads."""
    x = _f32(x).ravel()
    a, s, i, st = C.c_float(), C.c_double(), C.c_int32(), C.c_uint32(0)
    curve = np.empty(n_cand, dtype=np.float64) if want_curve else None
    _load().omse_oracle_activation_scale(_p(x, C.c_float), x.size, bits, int(is_signed), n_cand,
                                         _c32(hi_frac), refine_iters, C.byref(a), C.byref(s), C.byref(i),
                                         _p(curve, C.c_double), C.byref(st))
    return PhiResult(a.value, s.value, i.value, None, curve, st.value)


@dataclass
class ResidualResult:
    alpha: np.ndarray      # [n_tensors, S]
    sse: np.ndarray        # [n_tensors, S] float64: error after tensors 1..j
    best_idx: np.ndarray   # [n_tensors, S]
    codes: np.ndarray      # [n_tensors, S, K] int8
    status: int


def residual_rows(t, bits=(4, 4), is_signed=True, n_cand=1024, hi_frac=1.0, refine_iters=3,
                  n_sweeps=1) -> ResidualResult:
    """Algorithm 1 (Section 3.5) applied kernel-wise; n_sweeps=1 is the residual scheme of Section 3.7."""
    t = _f32(t)
    assert t.ndim == 2
    S, K = t.shape
    n = len(bits)
    b = (C.c_int * n)(*bits)
    alpha = np.zeros((n, S), np.float32)
    sse = np.zeros((n, S), np.float64)
    idx = np.zeros((n, S), np.int32)
    q = np.zeros((n, S, K), np.int8)
    st = C.c_uint32(0)
    _load().omse_oracle_residual_rows(_p(t, C.c_float), S, K, b, int(is_signed), n_cand, _c32(hi_frac),
                                      refine_iters, n, n_sweeps, _p(alpha, C.c_float), _p(sse, C.c_double),
                                      _p(idx, C.c_int32), _p(q, C.c_int8), C.byref(st))
    return ResidualResult(alpha, sse, idx, q, st.value)


def dual_scales(max_abs, hi_frac1, hi_frac2, n_cand1, n_cand2, c, d):
    a1, a2 = C.c_float(), C.c_float()
    _load().omse_oracle_dual_scales(_c32(max_abs), _c32(hi_frac1), _c32(hi_frac2), n_cand1, n_cand2, c, d,
                                    C.byref(a1), C.byref(a2))
    return a1.value, a2.value


def dual_sse_at(x, a1, a2, bits1=4, bits2=4, is_signed=True) -> float:
    """Section 3.5 dual objective at a given pair of scales (per-element enumeration of the first code)."""
    x = _f32(x).ravel()
    return float(_load().omse_oracle_dual_sse_at(_p(x, C.c_float), x.size, _c32(a1), _c32(a2), bits1, bits2,
                                                 int(is_signed)))


@dataclass
class DualResult:
    alpha: np.ndarray      # [2] or [2, S]
    sse: object            # float or [S] float64
    best_idx: object       # flat pair index c*C2+d
    codes: np.ndarray | None   # [2, K] or [2, S, K]
    sse_curve: np.ndarray | None
    status: int


def dual(x, bits1=4, bits2=4, is_signed=True, n_cand1=32, n_cand2=32, hi_frac1=1.0, hi_frac2=0.25, start_idx=-1,
         want_curve=False) -> DualResult:
    """Dual line search of Section 3.5 on one segment."""
    x = _f32(x).ravel()
    a = np.zeros(2, np.float32)
    s, i, st = C.c_double(), C.c_int32(), C.c_uint32(0)
    q = np.zeros((2, x.size), np.int8)
    curve = np.empty(n_cand1 * n_cand2, np.float64) if want_curve else None
    _load().omse_oracle_dual(_p(x, C.c_float), x.size, bits1, bits2, int(is_signed), n_cand1, n_cand2,
                             _c32(hi_frac1), _c32(hi_frac2), start_idx, _p(a, C.c_float), C.byref(s), C.byref(i),
                             _p(q[0], C.c_int8), _p(q[1], C.c_int8), _p(curve, C.c_double), C.byref(st))
    return DualResult(a, s.value, i.value, q, curve, st.value)


def dual_rows(t, bits1=4, bits2=4, is_signed=True, n_cand1=32, n_cand2=32, hi_frac1=1.0, hi_frac2=0.25,
              start_idx=None) -> DualResult:
    """Kernel-wise dual line search over the rows of a 2-D array."""
    t = _f32(t)
    S, K = t.shape
    alpha = np.zeros((2, S), np.float32)
    sse = np.zeros(S, np.float64)
    idx = np.zeros(S, np.int32)
    q = np.zeros((2, S, K), np.int8)
    st = C.c_uint32(0)
    si = None if start_idx is None else np.ascontiguousarray(start_idx, dtype=np.int32)
    _load().omse_oracle_dual_rows(_p(t, C.c_float), S, K, bits1, bits2, int(is_signed), n_cand1, n_cand2,
                                  _c32(hi_frac1), _c32(hi_frac2), _p(si, C.c_int32), _p(alpha, C.c_float),
                                  _p(sse, C.c_double), _p(idx, C.c_int32), _p(q, C.c_int8), C.byref(st))
    return DualResult(alpha, sse, idx, q, None, st.value)


def layer_mse(sse, kernel_len: int) -> float:
    """Section 3.5: MSE of a layer from its kernels' squared errors (fp32 values as the library outputs them)."""
    e = _f32(sse).ravel()
    return float(_load().omse_oracle_layer_mse(_p(e, C.c_float), e.size, kernel_len))


def compression_ratio(n_kernels, kernel_len, bits, n_tensors) -> float:
    n = len(n_kernels)
    a = (C.c_int64 * n)(*n_kernels)
    b = (C.c_int64 * n)(*kernel_len)
    c = (C.c_int * n)(*bits)
    d = (C.c_int * n)(*n_tensors)
    return float(_load().omse_oracle_compression_ratio(a, b, c, d, n))


def alg1_rows(t, bits=(4, 4), is_signed=(True, True), n_cand=1024, hi_frac=1.0, refine_iters=3, n_sweeps=2):
    """Algorithm 1 with one signedness flag per quantized tensor; also returns the error after every update
    as sse_sweeps [n_sweeps, n_tensors, S]."""
    t = _f32(t)
    S, K = t.shape
    n = len(bits)
    b = (C.c_int * n)(*bits)
    f = (C.c_int * n)(*[int(x) for x in is_signed])
    alpha = np.zeros((n, S), np.float32)
    sse = np.zeros((n, S), np.float64)
    idx = np.zeros((n, S), np.int32)
    q = np.zeros((n, S, K), np.int8)
    hist = np.zeros((n_sweeps, n, S), np.float64)
    st = C.c_uint32(0)
    _load().omse_oracle_alg1_rows(_p(t, C.c_float), S, K, b, f, n_cand, _c32(hi_frac), refine_iters, n, n_sweeps,
                                  _p(alpha, C.c_float), _p(sse, C.c_double), _p(idx, C.c_int32), _p(q, C.c_int8),
                                  _p(hist, C.c_double), C.byref(st))
    return ResidualResult(alpha, sse, idx, q, st.value), hist


@dataclass
class OffsetResult:
    alpha: np.ndarray
    delta: np.ndarray
    sse: np.ndarray
    best_idx: np.ndarray
    codes: np.ndarray
    status: int


def offset_rows(w, bits=4, n_cand=256, hi_frac=1.0, refine_iters=3, start_idx=None) -> OffsetResult:
    """Section 3.1 quantization with offset delta = min, scale by the MMSE search, row by row
    (a 1-row array is the per-tensor case)."""
    w = _f32(w)
    S, K = w.shape
    alpha, delta = np.empty(S, np.float32), np.empty(S, np.float32)
    sse, idx = np.empty(S, np.float64), np.empty(S, np.int32)
    q = np.empty((S, K), np.int8)
    st = C.c_uint32(0)
    si = None if start_idx is None else np.ascontiguousarray(start_idx, dtype=np.int32)
    _load().omse_oracle_offset_rows(_p(w, C.c_float), S, K, bits, n_cand, _c32(hi_frac), refine_iters,
                                    _p(si, C.c_int32), _p(alpha, C.c_float), _p(delta, C.c_float),
                                    _p(sse, C.c_double), _p(idx, C.c_int32), _p(q, C.c_int8), C.byref(st))
    return OffsetResult(alpha, delta, sse, idx, q, st.value)


SOLVER_UNIFORM, SOLVER_ALTERNATING, SOLVER_GOLDEN = 0, 1, 2


@dataclass
class SolverResult:
    alpha: np.ndarray
    sse: np.ndarray
    codes: np.ndarray
    status: int
    n_evals: int = 0


def solver_rows(w, solver, bits=4, is_signed=True, n_iter=20, hi_frac=1.0, refine_iters=0) -> SolverResult:
    """Comparison solvers of Section 3.4 (uniform / alternating / golden-section), row by row."""
    w = _f32(w)
    S, K = w.shape
    alpha, sse = np.empty(S, np.float32), np.empty(S, np.float64)
    q = np.empty((S, K), np.int8)
    st = C.c_uint32(0)
    _load().omse_oracle_solver_rows(_p(w, C.c_float), S, K, bits, int(is_signed), solver, n_iter, _c32(hi_frac),
                                    refine_iters, _p(alpha, C.c_float), _p(sse, C.c_double), _p(q, C.c_int8),
                                    C.byref(st))
    return SolverResult(alpha, sse, q, st.value)


def solver_phi(x, solver, bits=4, is_signed=True, n_iter=20, hi_frac=1.0, refine_iters=0) -> SolverResult:
    """One segment; also returns the number of objective evaluations the solver made."""
    x = _f32(x).ravel()
    a, s, n, st = C.c_float(), C.c_double(), C.c_int32(), C.c_uint32(0)
    q = np.empty(x.size, np.int8)
    _load().omse_oracle_solver_phi(_p(x, C.c_float), x.size, bits, int(is_signed), solver, n_iter, _c32(hi_frac),
                                   refine_iters, C.byref(a), C.byref(s), _p(q, C.c_int8), C.byref(n), C.byref(st))
    return SolverResult(a.value, s.value, q, st.value, n.value)


def affine_rows(w, bits=4, n_cand=256, hi_frac=1.0, n_delta=8, off_frac=0.25, refine_iters=3,
                start_flat=None) -> OffsetResult:
    """Offset scheme of Section 3.1 with offset and scale both searched on grids, row by row;
    best_idx is the flat index d*n_cand + c."""
    w = _f32(w)
    S, K = w.shape
    alpha, delta = np.empty(S, np.float32), np.empty(S, np.float32)
    sse, idx = np.empty(S, np.float64), np.empty(S, np.int32)
    q = np.empty((S, K), np.int8)
    st = C.c_uint32(0)
    si = None if start_flat is None else np.ascontiguousarray(start_flat, dtype=np.int32)
    _load().omse_oracle_affine_rows(_p(w, C.c_float), S, K, bits, n_cand, _c32(hi_frac), n_delta, _c32(off_frac),
                                    refine_iters, _p(si, C.c_int32), _p(alpha, C.c_float), _p(delta, C.c_float),
                                    _p(sse, C.c_double), _p(idx, C.c_int32), _p(q, C.c_int8), C.byref(st))
    return OffsetResult(alpha, delta, sse, idx, q, st.value)


def affine_phi(x, bits=4, n_cand=256, hi_frac=1.0, n_delta=8, off_frac=0.25, refine_iters=3, want_curve=False):
    """One segment; returns (alpha, delta, sse, flat best index, codes, curve [n_delta, n_cand] or None)."""
    x = _f32(x).ravel()
    a, d, s, i, st = C.c_float(), C.c_float(), C.c_double(), C.c_int32(), C.c_uint32(0)
    q = np.empty(x.size, np.int8)
    curve = np.empty((n_delta, n_cand), np.float64) if want_curve else None
    _load().omse_oracle_affine_phi(_p(x, C.c_float), x.size, bits, n_cand, _c32(hi_frac), n_delta, _c32(off_frac),
                                   refine_iters, -1, C.byref(a), C.byref(d), C.byref(s), C.byref(i),
                                   _p(q, C.c_int8), _p(curve, C.c_double), C.byref(st))
    return a.value, d.value, s.value, i.value, q, curve


def alg1_rows_eps(t, bits=(4, 4), is_signed=(True, True), n_cand=1024, hi_frac=1.0, refine_iters=3, max_sweeps=8,
                  eps=1e-3):
    """Algorithm 1 with its while-condition: sweeps go on while the relative decrease of the error over a
    sweep exceeds eps (at most max_sweeps).  Returns (result, history [max_sweeps, n, S], sweeps_done [S])."""
    t = _f32(t)
    S, K = t.shape
    n = len(bits)
    b = (C.c_int * n)(*bits)
    f = (C.c_int * n)(*[int(x) for x in is_signed])
    alpha = np.zeros((n, S), np.float32)
    sse = np.zeros((n, S), np.float64)
    idx = np.zeros((n, S), np.int32)
    q = np.zeros((n, S, K), np.int8)
    hist = np.zeros((max_sweeps, n, S), np.float64)
    done = np.zeros(S, np.int32)
    st = C.c_uint32(0)
    _load().omse_oracle_alg1_rows_eps(_p(t, C.c_float), S, K, b, f, n_cand, _c32(hi_frac), refine_iters, n,
                                      max_sweeps, float(eps), _p(alpha, C.c_float), _p(sse, C.c_double),
                                      _p(idx, C.c_int32), _p(q, C.c_int8), _p(hist, C.c_double), _p(done, C.c_int32),
                                      C.byref(st))
    return ResidualResult(alpha, sse, idx, q, st.value), hist, done


@dataclass
class KeyLayerResult:
    first: list            # RowsResult per layer (single quantized tensor)
    mse: np.ndarray        # [L] float64, from the fp32 per-kernel errors
    is_key: np.ndarray     # [L] bool
    second: dict           # layer index -> ResidualResult (two tensors) for the key layers
    compression_ratio: float


def key_layer_pipeline(layers, bits=4, is_signed=True, n_cand=1024, hi_frac=1.0, refine_iters=3,
                       tau=8e-5) -> KeyLayerResult:
    """Section 3.5 end to end on a list of 2-D weight arrays: quantize every layer, MSE per layer, layers with
    MSE > tau get a second quantized tensor (the residual scheme, one sweep), compression ratio of the result.
    Only an ordering of calls to the functions above."""
    first = [quantize_rows(w, bits, is_signed, n_cand, hi_frac, refine_iters) for w in layers]
    mse = np.array([layer_mse(r.sse.astype(np.float32), w.shape[1]) for r, w in zip(first, layers)])
    is_key = mse > float(np.float32(tau))
    second = {l: residual_rows(layers[l], (bits, bits), is_signed, n_cand, hi_frac, refine_iters, 1)
              for l in np.nonzero(is_key)[0]}
    cr = compression_ratio([w.shape[0] for w in layers], [w.shape[1] for w in layers], [bits] * len(layers),
                           [2 if k else 1 for k in is_key])
    return KeyLayerResult(first, mse, is_key, second, cr)


def pack_int4(codes_) -> np.ndarray:
    q = np.ascontiguousarray(codes_, dtype=np.int8).ravel()
    out = np.empty((q.size + 1) // 2, np.uint8)
    _load().omse_oracle_pack_int4(_p(q, C.c_int8), q.size, _p(out, C.c_uint8))
    return out


def unpack_int4(packed, n: int, is_signed: bool) -> np.ndarray:
    p = np.ascontiguousarray(packed, dtype=np.uint8).ravel()
    out = np.empty(n, np.int8)
    _load().omse_oracle_unpack_int4(_p(p, C.c_uint8), n, int(is_signed), _p(out, C.c_int8))
    return out
