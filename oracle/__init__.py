"""CPU oracle for the GEMM hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference
legs may import this package.  It shares no code with the CUDA path and does not
import it.  The arithmetic lives in ``oracle_gemm.c`` (a plain fp64 triple loop
following the BLAS definition the paper's Section 6 compares against); this
file builds that C file with gcc, wraps it with ctypes, and adds the acceptance
metric and a whole-matrix Freivalds check written with numpy.

Parity status: pinned for finite inputs (see tests/test_oracle_pins.py);
behaviour on Inf/NaN operands is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_gemm.c")
_LIB = os.path.join(_HERE, "liboracle_gemm.so")

BF16, FP16, FP32 = 0, 1, 2
ROW_MAJOR, COL_MAJOR = 0, 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the library is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        common = [i64, i64, i64, vp, vp, vp, ci, ci, ci, ci, ci, i64, i64, i64, dbl, dbl]
        _lib.oracle_gemm.argtypes = common + [vp, vp]
        _lib.oracle_gemm.restype = ci
        _lib.oracle_gemm_rows.argtypes = common + [i64, i64, vp, vp]
        _lib.oracle_gemm_rows.restype = ci
        _lib.oracle_gemm_entries.argtypes = common + [i64, vp, vp, vp, vp]
        _lib.oracle_gemm_entries.restype = ci
        _lib.oracle_gemv.argtypes = [i64, i64, vp, i64, vp, vp, dbl, dbl, vp, vp]
        _lib.oracle_gemv.restype = ci
        _lib.oracle_gemv_colmajor.argtypes = [i64, i64, vp, i64, vp, vp, dbl, dbl, vp, vp]
        _lib.oracle_gemv_colmajor.restype = ci
        _lib.oracle_widen.argtypes = [ctypes.c_uint32, ci]
        _lib.oracle_widen.restype = dbl
        _lib.oracle_num_threads.restype = ci
        _lib.oracle_set_num_threads.argtypes = [ci]
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(int(n))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_buf(buf, dtype, n_needed, what):  # dtype FP32 also covers tf32-mode operands (stored as float32)
    want = np.float32 if dtype == FP32 else np.uint16
    if buf.dtype != want or not buf.flags.c_contiguous or buf.ndim != 1:
        raise ValueError(f"{what}: need flat contiguous {want.__name__}")
    if buf.size < n_needed:
        raise ValueError(f"{what}: buffer too small ({buf.size} < {n_needed})")


def _common(M, N, K, A, B, Cin, ab_dtype, c_dtype, a_layout, b_layout, c_layout, lda, ldb, ldc,
            alpha, beta):
    _check_buf(A, ab_dtype, (M if a_layout == ROW_MAJOR else K) * lda if M and K else 0, "A")
    _check_buf(B, ab_dtype, (K if b_layout == ROW_MAJOR else N) * ldb if K and N else 0, "B")
    if beta != 0.0:
        if Cin is None:
            raise ValueError("beta != 0 needs C_in")
        _check_buf(Cin, c_dtype, (M if c_layout == ROW_MAJOR else N) * ldc if M and N else 0, "C")
    return [M, N, K, _ptr(A), _ptr(B), _ptr(Cin) if beta != 0.0 else None, ab_dtype, c_dtype,
            a_layout, b_layout, c_layout, lda, ldb, ldc, float(alpha), float(beta)]


def gemm(M, N, K, A, B, Cin, ab_dtype, c_dtype, a_layout, b_layout, c_layout, lda, ldb, ldc,
         alpha, beta, rows=None):
    """Reference result and metric denominator, both (rows x N) float64, row-major.

    ``rows=(r0, r1)`` restricts the evaluation to a row band of C.
    """
    r0, r1 = (0, M) if rows is None else rows
    cref = np.empty((r1 - r0, N), dtype=np.float64)
    den = np.empty((r1 - r0, N), dtype=np.float64)
    args = _common(M, N, K, A, B, Cin, ab_dtype, c_dtype, a_layout, b_layout, c_layout,
                   lda, ldb, ldc, alpha, beta)
    rc = lib().oracle_gemm_rows(*args, r0, r1, _ptr(cref), _ptr(den))
    if rc != 0:
        raise RuntimeError(f"oracle_gemm_rows failed with code {rc}")
    return cref, den


def gemm_entries(M, N, K, A, B, Cin, ab_dtype, c_dtype, a_layout, b_layout, c_layout, lda, ldb, ldc,
                 alpha, beta, rows, cols):
    """Reference result and denominator for the listed (row, col) entries."""
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    cref = np.empty(rows.size, dtype=np.float64)
    den = np.empty(rows.size, dtype=np.float64)
    args = _common(M, N, K, A, B, Cin, ab_dtype, c_dtype, a_layout, b_layout, c_layout,
                   lda, ldb, ldc, alpha, beta)
    rc = lib().oracle_gemm_entries(*args, rows.size, _ptr(rows), _ptr(cols), _ptr(cref), _ptr(den))
    if rc != 0:
        raise RuntimeError(f"oracle_gemm_entries failed with code {rc}")
    return cref, den


def gemv(M, N, A, lda, x, y, alpha, beta, layout=ROW_MAJOR):
    """Reference y and metric denominator (float64, length M) of the fp32 GEMV, A row- or column-major."""
    a_need = ((M - 1) * lda + N if layout == ROW_MAJOR else (N - 1) * lda + M) if M and N else 0
    for buf, need, what in ((A, a_need, "A"), (x, N, "x"), (y, M, "y")):
        if buf.dtype != np.float32 or not buf.flags.c_contiguous or buf.size < need:
            raise ValueError(f"{what}: need contiguous float32 of at least {need} elements")
    yref = np.empty(M, dtype=np.float64)
    den = np.empty(M, dtype=np.float64)
    fn = lib().oracle_gemv if layout == ROW_MAJOR else lib().oracle_gemv_colmajor
    rc = fn(M, N, _ptr(A), lda, _ptr(x), _ptr(y), float(alpha), float(beta), _ptr(yref), _ptr(den))
    if rc != 0:
        raise RuntimeError(f"oracle_gemv failed with code {rc}")
    return yref, den


def gemm_problem(p, rows=None):
    """``gemm`` on an object with the descriptor fields and host buffers A, B, C."""
    return gemm(p.M, p.N, p.K, p.A, p.B, p.C, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout,
                p.c_layout, p.lda, p.ldb, p.ldc, p.alpha, p.beta, rows=rows)


def gemm_problem_entries(p, rows, cols):
    return gemm_entries(p.M, p.N, p.K, p.A, p.B, p.C, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout,
                        p.c_layout, p.lda, p.ldb, p.ldc, p.alpha, p.beta, rows, cols)


# ----------------------------------------------------------------------------
# widening of stored values (numpy; used by the metric and the Freivalds check)
# ----------------------------------------------------------------------------
def widen(buf: np.ndarray, dtype: int) -> np.ndarray:
    """Stored values -> float64, exactly."""
    if dtype == FP32:
        return buf.astype(np.float64)
    if dtype == FP16:
        return buf.view(np.float16).astype(np.float64)
    if dtype == BF16:
        return (buf.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    raise ValueError(dtype)


def logical_view(buf, rows, cols, layout, ld, dtype):
    """Float64 logical rows x cols matrix read through the layout accessor."""
    outer, inner = (rows, cols) if layout == ROW_MAJOR else (cols, rows)
    v = widen(buf[: outer * ld].reshape(outer, ld)[:, :inner], dtype)
    return v if layout == ROW_MAJOR else v.T


# ----------------------------------------------------------------------------
# acceptance metric
# ----------------------------------------------------------------------------
TOLERANCE = 1e-3


def error_ratio(c_got: np.ndarray, cref: np.ndarray, den: np.ndarray) -> np.ndarray:
    """|C - Cref| / Den element-wise; 0/0 := 0, x/0 := inf for x != 0.

    Den is the oracle's sum_k |a_ik b_kj| + |beta c_ij| (no alpha factor: the
    literal acceptance formula).
    """
    num = np.abs(np.asarray(c_got, dtype=np.float64) - cref)
    out = np.empty_like(num)
    zero = den == 0.0
    np.divide(num, den, out=out, where=~zero)
    out[zero] = np.where(num[zero] == 0.0, 0.0, np.inf)
    out[np.isnan(num)] = np.inf
    return out


def max_error(c_got, cref, den) -> float:
    r = error_ratio(c_got, cref, den)
    return float(r.max()) if r.size else 0.0


def output_rounding_slack(cref: np.ndarray, c_dtype: int) -> np.ndarray:
    """Half an ulp of the output type relative to |Cref| (0 for fp32 output).

    The acceptance formula has no term for rounding the result into a 16-bit
    output; where |Cref| is close to Den (same-sign data) a correctly rounded
    bf16 result can exceed 1e-3 * Den.  Closed-form tests on such data use the
    widened gate |dC| <= 1e-3 * Den + u_out * |Cref|.
    """
    u = {FP32: 0.0, BF16: 2.0 ** -8, FP16: 2.0 ** -11}[c_dtype]
    slack = u * np.abs(cref)
    if c_dtype != FP32:
        # Below the smallest normal number the spacing of the output type no longer shrinks with the value
        # (gradual underflow: 2^-24 for fp16 below 2^-14, 2^-133 for bf16 below 2^-126), so half an ulp is a
        # constant there.  Zero is representable: no slack at Cref == 0.
        min_normal, half_spacing = {BF16: (2.0 ** -126, 2.0 ** -134), FP16: (2.0 ** -14, 2.0 ** -25)}[c_dtype]
        a = np.abs(cref)
        slack = np.where((a > 0) & (a < min_normal), half_spacing, slack)
    return slack


# ----------------------------------------------------------------------------
# Freivalds whole-matrix check
# ----------------------------------------------------------------------------
def freivalds(p, c_got: np.ndarray, n_vectors: int = 4, seed: int = 12345):
    """Compare C_got @ x with alpha*A(Bx) + beta*C_in x for random +-1 vectors x.

    ``c_got`` is the logical M x N result in float64.  Returns the maximum over
    rows and vectors of |lhs - rhs| / bound with
    bound_i = (|A| (|B| |x|) + |beta| |C_in| |x|)_i, i.e. the row sum of the
    per-entry denominators; a value <= TOLERANCE is implied by every entry
    meeting the per-entry gate.  O(MN + MK + KN) work.
    """
    rng = np.random.default_rng(seed)
    A = logical_view(p.A, p.M, p.K, p.a_layout, p.lda, p.ab_dtype)
    B = logical_view(p.B, p.K, p.N, p.b_layout, p.ldb, p.ab_dtype)
    Cin = logical_view(p.C, p.M, p.N, p.c_layout, p.ldc, p.c_dtype) if p.beta != 0.0 else None
    absA, absB = np.abs(A), np.abs(B)
    worst = 0.0
    for _ in range(n_vectors):
        x = rng.integers(0, 2, size=p.N).astype(np.float64) * 2.0 - 1.0
        rhs = p.alpha * (A @ (B @ x))
        bound = absA @ (absB @ np.abs(x))
        if Cin is not None:
            rhs = rhs + p.beta * (Cin @ x)
            bound = bound + abs(p.beta) * (np.abs(Cin) @ np.abs(x))
        lhs = c_got @ x
        num = np.abs(lhs - rhs)
        ratio = np.where(bound > 0, num / np.where(bound > 0, bound, 1.0), np.where(num == 0, 0.0, np.inf))
        worst = max(worst, float(ratio.max()))
    return worst
