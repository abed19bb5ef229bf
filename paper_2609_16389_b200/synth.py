"""Seeded synthetic GEMM inputs (host side, numpy only).

This module serves both the CUDA path's harness and the CPU oracle's tests.  It
holds no GEMM arithmetic: it only draws matrix entries from a counter-based
generator, rounds them to the 16-bit storage type and lays them out in memory.

The paper's evaluation (Section 6, "Evaluation") uses dense matrices filled by
an integer hash; its exact hash is not reproduced here.  What matters for this
build is the same structure: dense, i.i.d., value of an entry a pure function
of (seed, matrix tag, row, column), so the same logical matrix can be stored in
any layout or leading dimension.

Entry recipe
------------
* ``uniform``: u = (h >> 40) / 2**23 - 1 with h a 64-bit hash, i.e. a point of
  the 2**24-point grid on [-1, 1); exactly representable in fp32, then rounded
  to nearest-even into bf16 or fp16 (so both -1.0 and +1.0 occur after
  rounding).
* ``normal``: Box-Muller in fp64 from two grid uniforms on (0, 1], then rounded
  to nearest-even into the storage type.
"""
from __future__ import annotations

import os

import numpy as np

BASE_SEED = 260916389
TAG_A, TAG_B, TAG_C = 1, 2, 3

BF16, FP16, FP32 = 0, 1, 2
ROW_MAJOR, COL_MAJOR = 0, 1

_DTYPE_NAMES = {BF16: "bf16", FP16: "fp16", FP32: "fp32"}
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def dtype_name(code: int) -> str:
    return _DTYPE_NAMES[code]


def elem_size(code: int) -> int:
    return 4 if code == FP32 else 2


# ----------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------
def _mix64(x: np.ndarray) -> np.ndarray:
    """A 64-bit finaliser (xor-shift / odd-multiply rounds); x is uint64."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= np.uint64(0xBF58476D1CE4E5B9)
    x ^= x >> np.uint64(27)
    x *= np.uint64(0x94D049BB133111EB)
    x ^= x >> np.uint64(31)
    return x


def _hash_grid(seed: int, tag: int, stream: int, rows: np.ndarray, cols: np.ndarray) -> np.ndarray:
    """64-bit hash of (seed, tag, stream, i, j) for the outer grid rows x cols."""
    with np.errstate(over="ignore"):
        s = np.uint64((seed * 0x9E3779B97F4A7C15 + tag * 0xD1B54A32D192ED03
                       + stream * 0x8CB92BA72F3D8DD7) & 0xFFFFFFFFFFFFFFFF)
        ri = _mix64(rows.astype(np.uint64) * np.uint64(0x9E3779B97F4A7C15) + s)
        cj = cols.astype(np.uint64) * np.uint64(0xC2B2AE3D27D4EB4F) + np.uint64(0x165667B19E3779F9)
        h = ri[:, None] ^ cj[None, :]
        return _mix64(h + s)


def uniform_pm1(seed: int, tag: int, rows: np.ndarray, cols: np.ndarray, stream: int = 0) -> np.ndarray:
    """Grid uniforms on [-1, 1) as float32 (exact), shape (len(rows), len(cols))."""
    h = _hash_grid(seed, tag, stream, rows, cols)
    k = (h >> np.uint64(40)).astype(np.int64)          # 24 bits
    return ((k - (1 << 23)).astype(np.float32)) * np.float32(2.0 ** -23)


def _uniform_01_open_low(seed: int, tag: int, rows, cols, stream: int) -> np.ndarray:
    """Grid uniforms on (0, 1] as float64."""
    h = _hash_grid(seed, tag, stream, rows, cols)
    k = (h >> np.uint64(40)).astype(np.float64)
    return (k + 1.0) * 2.0 ** -24


def normal_01(seed: int, tag: int, rows: np.ndarray, cols: np.ndarray) -> np.ndarray:
    """Standard normals (float64) by Box-Muller from two independent streams."""
    u1 = _uniform_01_open_low(seed, tag, rows, cols, 1)
    u2 = _uniform_01_open_low(seed, tag, rows, cols, 2)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


# ----------------------------------------------------------------------------
# storage rounding (round-to-nearest-even)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even, finite inputs."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = b + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def to_fp16_bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x).astype(np.float16).view(np.uint16)


def f32_round_to_tf32(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to nearest-even onto the tf32 grid (10 fraction bits), still stored as fp32."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(13)) & np.uint32(1)
    r = (b + np.uint32(0x0FFF) + lsb) & np.uint32(0xFFFFE000)
    return r.view(np.float32)


def round_to_storage(x: np.ndarray, dtype: int, operand: bool = False) -> np.ndarray:
    """Round a real array to the storage type; returns uint16 bits or float32.

    ``operand=True`` with FP32 means an A or B matrix of the tf32 mode: stored as fp32, with values
    on the tf32 grid, so that the tensor core (which ignores the low 13 fraction bits) and the oracle
    (which widens the stored value exactly) see the same numbers.
    """
    if dtype == FP32 and operand:
        return f32_round_to_tf32(x.astype(np.float32))
    if dtype == BF16:
        return f32_to_bf16_bits(x.astype(np.float32))
    if dtype == FP16:
        return to_fp16_bits(x)
    if dtype == FP32:
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(f"bad dtype {dtype}")


def storage_np_dtype(dtype: int):
    return np.float32 if dtype == FP32 else np.uint16


# ----------------------------------------------------------------------------
# layouts
# ----------------------------------------------------------------------------
def min_ld(rows: int, cols: int, layout: int) -> int:
    return cols if layout == ROW_MAJOR else rows


def buffer_elems(rows: int, cols: int, layout: int, ld: int) -> int:
    return (rows if layout == ROW_MAJOR else cols) * ld


def store(logical: np.ndarray, layout: int, ld: int | None = None, pad=None) -> np.ndarray:
    """Lay a logical rows x cols array out as a flat buffer with leading dimension ld.

    Padding elements (ld beyond the extent) are filled with ``pad`` (same storage
    type as ``logical``); default zero bits.
    """
    rows, cols = logical.shape
    if ld is None:
        ld = min_ld(rows, cols, layout)
    if ld < min_ld(rows, cols, layout):
        raise ValueError("ld below extent")
    outer, inner = (rows, cols) if layout == ROW_MAJOR else (cols, rows)
    buf = np.empty((outer, ld), dtype=logical.dtype)
    if ld > inner:
        buf[:, inner:] = 0 if pad is None else pad
    buf[:, :inner] = logical if layout == ROW_MAJOR else logical.T
    return buf.reshape(-1)


def load(buf: np.ndarray, rows: int, cols: int, layout: int, ld: int) -> np.ndarray:
    """Inverse of ``store``: the logical rows x cols view (a copy)."""
    outer, inner = (rows, cols) if layout == ROW_MAJOR else (cols, rows)
    v = buf.reshape(outer, ld)[:, :inner]
    return np.array(v if layout == ROW_MAJOR else v.T)


# ----------------------------------------------------------------------------
# matrices and workloads
# ----------------------------------------------------------------------------
def matrix(seed: int, tag: int, rows: int, cols: int, dtype: int, dist: str = "uniform",
           chunk_rows: int = 512, operand: bool = False) -> np.ndarray:
    """Logical rows x cols matrix in storage type (uint16 bits, or float32).

    An entry depends on (seed, tag, row, column) only, so row blocks are filled by a few threads side
    by side (numpy releases the interpreter lock inside its array operations)."""
    if dist not in ("uniform", "normal"):
        raise ValueError(dist)
    out = np.empty((rows, cols), dtype=storage_np_dtype(dtype))
    cj = np.arange(cols, dtype=np.int64)

    def fill(r0):
        ri = np.arange(r0, min(rows, r0 + chunk_rows), dtype=np.int64)
        x = uniform_pm1(seed, tag, ri, cj) if dist == "uniform" else normal_01(seed, tag, ri, cj)
        out[r0:r0 + len(ri)] = round_to_storage(x, dtype, operand)

    starts = range(0, rows, chunk_rows)
    threads = min(len(starts), os.cpu_count() or 1, 32)
    if threads <= 1 or rows * cols < (1 << 20):
        for r0 in starts:
            fill(r0)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, starts))
    return out


def shape_seed(M: int, N: int, K: int) -> int:
    """Per-shape seed for the shape sweep."""
    x = np.array([BASE_SEED * 1000003 + M * 2654435761 + N * 40503 + K * 2246822519], dtype=np.uint64)
    return int(_mix64(x)[0] & np.uint64(0x7FFFFFFF))


class Problem:
    """One GEMM problem: descriptor fields plus host buffers (flat numpy arrays)."""

    def __init__(self, name, M, N, K, ab_dtype, c_dtype, a_layout, b_layout, c_layout,
                 alpha, beta, seed, dist="uniform", lda=None, ldb=None, ldc=None):
        self.name = name
        self.M, self.N, self.K = M, N, K
        self.ab_dtype, self.c_dtype = ab_dtype, c_dtype
        self.a_layout, self.b_layout, self.c_layout = a_layout, b_layout, c_layout
        self.alpha, self.beta = float(alpha), float(beta)
        self.seed, self.dist = seed, dist
        self.lda = lda if lda is not None else max(1, min_ld(M, K, a_layout))
        self.ldb = ldb if ldb is not None else max(1, min_ld(K, N, b_layout))
        self.ldc = ldc if ldc is not None else max(1, min_ld(M, N, c_layout))
        self.A = self.B = self.C = None
        # fp32 operands (tf32 math): True draws A and B on the tf32 grid (10 fraction bits), False keeps
        # the full 24-bit significands of the draw
        self.tf32_grid = True

    def generate(self, pad_a=None, pad_b=None, pad_c=None):
        """Fill A, B and C_in.  C_in is drawn uniform[-1,1] in every case (it is
        only read when beta != 0)."""
        a = matrix(self.seed, TAG_A, self.M, self.K, self.ab_dtype, self.dist, operand=self.tf32_grid)
        b = matrix(self.seed, TAG_B, self.K, self.N, self.ab_dtype, self.dist, operand=self.tf32_grid)
        c = matrix(self.seed, TAG_C, self.M, self.N, self.c_dtype, "uniform")
        self.A = store(a, self.a_layout, self.lda, pad_a)
        self.B = store(b, self.b_layout, self.ldb, pad_b)
        self.C = store(c, self.c_layout, self.ldc, pad_c)
        return self

    @property
    def flop(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> int:
        """Each operand once, C out once, C in once iff beta != 0."""
        ab = elem_size(self.ab_dtype)
        cb = elem_size(self.c_dtype)
        n = ab * (self.M * self.K + self.K * self.N) + cb * self.M * self.N
        if self.beta != 0.0:
            n += cb * self.M * self.N
        return n


class BatchedProblem(Problem):
    """`batch` independent problems of one shape, packed back to back (strides = one matrix)."""

    def __init__(self, name, batch, *args, **kw):
        super().__init__(name, *args, **kw)
        self.batch = batch
        self.stride_a = self.stride_b = self.stride_c = 0

    def generate(self, **kw):
        parts = []
        base_seed = self.seed
        for i in range(self.batch):
            self.seed = base_seed + 7919 * i
            super().generate(**kw)
            parts.append((self.A, self.B, self.C))
        self.seed = base_seed
        self.stride_a, self.stride_b, self.stride_c = parts[0][0].size, parts[0][1].size, parts[0][2].size
        self.A = np.concatenate([q[0] for q in parts])
        self.B = np.concatenate([q[1] for q in parts])
        self.C = np.concatenate([q[2] for q in parts])
        return self

    def matrix(self, i: int) -> Problem:
        """Problem view of matrix i (shares the packed buffers)."""
        q = Problem(f"{self.name}[{i}]", self.M, self.N, self.K, self.ab_dtype, self.c_dtype, self.a_layout,
                    self.b_layout, self.c_layout, self.alpha, self.beta, self.seed, self.dist,
                    self.lda, self.ldb, self.ldc)
        q.A = self.A[i * self.stride_a:(i + 1) * self.stride_a]
        q.B = self.B[i * self.stride_b:(i + 1) * self.stride_b]
        q.C = self.C[i * self.stride_c:(i + 1) * self.stride_c]
        return q

    @property
    def flop(self) -> float:
        return self.batch * super().flop

    @property
    def algorithmic_bytes(self) -> int:
        return self.batch * super().algorithmic_bytes


def batched(batch: int, n: int) -> BatchedProblem:
    """Strided batch of `batch` cubes n^3: bf16 uniform, A row / B col, bf16 C (the paper's
    evaluation also measures a strided-batched GEMM; it gives no sizes)."""
    return BatchedProblem(f"batched_{batch}x{n}", batch, n, n, n, BF16, BF16, ROW_MAJOR, COL_MAJOR, ROW_MAJOR,
                          1.0, 0.0, BASE_SEED + 50)


def tf32_square(n: int) -> Problem:
    """n^3 GEMM in the precision the paper measured (Section 6): fp32 storage, tf32 math, fp32 C."""
    return Problem(f"tf32_{n}", n, n, n, FP32, FP32, ROW_MAJOR, COL_MAJOR, ROW_MAJOR, 1.0, 0.0, BASE_SEED + 60)


def config(idx: int, variant: str | None = None) -> Problem:
    """The benchmark configurations (0-based index into the configuration list).

    0: 256^3 bf16, A row / B col, fp32 C, alpha=1 beta=0
    1: 4096^3 bf16, A row / B col, bf16 C, alpha=1 beta=0
    2: 8192^3 fp16 normal(0,1), A row / B row, fp32 C, alpha=0.5 beta=1, C_in uniform
    3: skinny 16384x1024x4096 (variant 'a') and 1024x16384x4096 (variant 'b'), bf16 -> bf16
    """
    seed = BASE_SEED + idx + 1
    if idx == 0:
        return Problem("cfg1_256", 256, 256, 256, BF16, FP32, ROW_MAJOR, COL_MAJOR, ROW_MAJOR, 1.0, 0.0, seed)
    if idx == 1:
        return Problem("cfg2_4096", 4096, 4096, 4096, BF16, BF16, ROW_MAJOR, COL_MAJOR, ROW_MAJOR, 1.0, 0.0, seed)
    if idx == 2:
        return Problem("cfg3_8192", 8192, 8192, 8192, FP16, FP32, ROW_MAJOR, ROW_MAJOR, ROW_MAJOR, 0.5, 1.0,
                       seed, dist="normal")
    if idx == 3:
        if variant in (None, "a"):
            return Problem("cfg4a_skinny", 16384, 1024, 4096, BF16, BF16, ROW_MAJOR, COL_MAJOR, ROW_MAJOR,
                           1.0, 0.0, seed)
        return Problem("cfg4b_skinny", 1024, 16384, 4096, BF16, BF16, ROW_MAJOR, COL_MAJOR, ROW_MAJOR,
                       1.0, 0.0, seed + 100)
    raise ValueError(idx)


SWEEP_DIMS = (512, 1000, 2048, 3072, 6144, 12288)


def sweep_problem(M: int, N: int, K: int) -> Problem:
    """One shape of the shape sweep: bf16 uniform, A row / B col, fp32 C."""
    return Problem(f"sweep_{M}x{N}x{K}", M, N, K, BF16, FP32, ROW_MAJOR, COL_MAJOR, ROW_MAJOR,
                   1.0, 0.0, shape_seed(M, N, K))
