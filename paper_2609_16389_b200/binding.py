"""ctypes binding of the C-ABI GEMM library (argument marshalling only).

Every function here has the name of the C entry point it calls; all compute
happens in the CUDA kernels behind ``exo_gemm_run``.  There is no fallback: if
the shared library cannot be built or loaded, importing ``lib()`` raises.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

OK, ERR_NULL, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(8)
BF16, FP16, FP32 = 0, 1, 2
ROW_MAJOR, COL_MAJOR = 0, 1

EXPORTED_SYMBOLS = (
    "exo_gemm_validate", "exo_gemm_create", "exo_gemm_run", "exo_gemm_check", "exo_gemm_plan_preview",
    "exo_gemm_get_info", "exo_gemm_destroy", "exo_gemm_status_string", "exo_gemm_last_cuda_error",
    "exo_gemm_schedule_enumerate", "exo_gemm_debug_set", "exo_gemm_run_static", "exo_gemm_schedule_work",
    "exo_gemm_create_batched", "exo_gemv_run", "exo_gemm_has_shared_operand_clusters", "exo_gemv_run_colmajor",
)


def flag_cta_group(g): return g & 3
def flag_tile_n(n): return ((n // 64) & 15) << 2
def flag_band(b): return (b & 15) << 6
FLAG_BANDS_ALONG_M = 1 << 10
FLAG_SPLIT_REDUCE_ADD = 1 << 11
def flag_grid_limit(c): return (c & 255) << 12
def flag_k_subblocks(k): return (k & 3) << 20
def flag_epi_buffers(b): return (b & 3) << 22
def flag_max_stages(s): return (s & 15) << 24
def flag_split_k(f): return (f & 15) << 28
FLAG2_SHARE_AUTO, FLAG2_SHARE_NEVER, FLAG2_SHARE_ALWAYS, FLAG2_SHARE_SUBSTITUTED = 0, 1, 2, 3
FLAG2_LEAN_AUTO, FLAG2_LEAN_NEVER, FLAG2_LEAN_ALWAYS = 0, 1 << 4, 2 << 4
def flag2_cta_rows(r): return ((r // 128) & 3) << 2


class Desc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("ab_dtype", ctypes.c_int32), ("c_dtype", ctypes.c_int32),
                ("a_layout", ctypes.c_int32), ("b_layout", ctypes.c_int32), ("c_layout", ctypes.c_int32),
                ("device", ctypes.c_int32),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64),
                ("flags", ctypes.c_uint32), ("flags2", ctypes.c_uint32)]


class Info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "cta_group", "tile_m", "tile_n", "tile_k", "stages", "grid", "smem_bytes", "tmem_columns",
        "tiles_m", "tiles_n", "raster_along_m", "raster_band", "swapped", "sm_count",
        "kernel_launches_per_run", "epilogue_buffers", "split_k", "tail_tiles", "workspace_bytes",
        "batch_count", "cluster_size", "tail_workers", "stages_direct", "lean_kernel", "repacked")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class ExoGemmError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {exo_gemm_status_string(status)} (status {status}, "
                         f"cuda error {exo_gemm_last_cuda_error()})")


_lib = None


def lib():
    """Loads (building first if needed) the CUDA library; raises if that fails."""
    global _lib
    if _lib is None:
        # EXO_GEMM_LIBRARY overrides (a development build); otherwise the variant library -- the base
        # library plus the shared-operand cluster kernels -- where its sources are present, else the base one
        # (a rank of a multi-GPU job always gets the base library)
        path = os.environ.get("EXO_GEMM_LIBRARY") or _build.build_preferred()
        if _build.multi_gpu_job() and os.path.basename(path) == os.path.basename(_build.SHARE_LIB):
            raise RuntimeError("the shared-operand cluster library is for single-GPU programs only")
        if not os.path.exists(path):
            raise RuntimeError("libexo_gemm.so is missing: the CUDA path cannot run")
        L = ctypes.CDLL(path)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.exo_gemm_validate.argtypes = [ctypes.POINTER(Desc)]
        L.exo_gemm_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Desc)]
        L.exo_gemm_run.argtypes = [vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp]
        L.exo_gemm_create_batched.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Desc), i64, i64, i64, i64]
        L.exo_gemm_create_batched.restype = ctypes.c_int
        L.exo_gemm_check.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        L.exo_gemm_plan_preview.argtypes = [ctypes.POINTER(Desc), i32, ctypes.POINTER(Info)]
        L.exo_gemm_get_info.argtypes = [vp, ctypes.POINTER(Info)]
        L.exo_gemm_destroy.argtypes = [vp]
        L.exo_gemm_status_string.argtypes = [ctypes.c_int]
        L.exo_gemm_status_string.restype = ctypes.c_char_p
        L.exo_gemm_last_cuda_error.restype = ctypes.c_int
        L.exo_gemm_has_shared_operand_clusters.restype = i32
        L.exo_gemm_schedule_enumerate.argtypes = [i32, i32, i32, i32, i32, i32, ctypes.POINTER(i32),
                                                  ctypes.POINTER(i32), i64]
        L.exo_gemm_schedule_enumerate.restype = i64
        L.exo_gemm_debug_set.argtypes = [vp, i32, i64]
        L.exo_gemv_run.argtypes = [i64, i64, vp, i64, vp, vp, ctypes.c_float, ctypes.c_float, vp]
        L.exo_gemv_run.restype = ctypes.c_int
        L.exo_gemv_run_colmajor.argtypes = [i64, i64, vp, i64, vp, vp, ctypes.c_float, ctypes.c_float, vp]
        L.exo_gemv_run_colmajor.restype = ctypes.c_int
        L.exo_gemm_schedule_work.argtypes = [i64, i32, i32, i32, i32, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i32),
                                             ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32), i64]
        L.exo_gemm_schedule_work.restype = i64
        L.exo_gemm_run_static.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, ctypes.c_float, ctypes.c_float, vp,
                                          ctypes.POINTER(ctypes.c_uint32)]
        L.exo_gemm_run_static.restype = ctypes.c_int
        for name in ("exo_gemm_validate", "exo_gemm_create", "exo_gemm_run", "exo_gemm_check",
                     "exo_gemm_plan_preview", "exo_gemm_get_info", "exo_gemm_destroy", "exo_gemm_debug_set"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def make_desc(M, N, K, ab_dtype, c_dtype, a_layout, b_layout, c_layout, lda=None, ldb=None, ldc=None,
              device=-1, flags=0, flags2=0) -> Desc:
    def ext(layout, rows, cols):
        return max(1, cols if layout == ROW_MAJOR else rows)
    return Desc(M, N, K, ab_dtype, c_dtype, a_layout, b_layout, c_layout, device,
                ext(a_layout, M, K) if lda is None else lda,
                ext(b_layout, K, N) if ldb is None else ldb,
                ext(c_layout, M, N) if ldc is None else ldc, flags, flags2)


# ---- one function per C entry point -------------------------------------------------
def exo_gemm_has_shared_operand_clusters() -> int:
    return int(lib().exo_gemm_has_shared_operand_clusters())


def exo_gemm_validate(desc: Desc) -> int:
    return lib().exo_gemm_validate(ctypes.byref(desc) if desc is not None else None)


def exo_gemm_create(desc: Desc):
    h = ctypes.c_void_p()
    st = lib().exo_gemm_create(ctypes.byref(h), ctypes.byref(desc))
    return st, (h if st == OK else None)


def exo_gemm_create_batched(desc: Desc, batch_count: int, stride_a: int, stride_b: int, stride_c: int):
    h = ctypes.c_void_p()
    st = lib().exo_gemm_create_batched(ctypes.byref(h), ctypes.byref(desc), batch_count, stride_a, stride_b, stride_c)
    return st, (h if st == OK else None)


def exo_gemm_run(handle, a_ptr: int, b_ptr: int, c_ptr: int, alpha: float, beta: float, stream: int = 0) -> int:
    return lib().exo_gemm_run(handle, a_ptr, b_ptr, c_ptr, alpha, beta, stream)


def exo_gemm_check(handle):
    detail = (ctypes.c_uint32 * 8)()
    st = lib().exo_gemm_check(handle, detail)
    return st, list(detail)


def exo_gemm_plan_preview(desc: Desc, sm_count: int):
    info = Info()
    st = lib().exo_gemm_plan_preview(ctypes.byref(desc), sm_count, ctypes.byref(info))
    return st, info


def exo_gemm_get_info(handle) -> Info:
    info = Info()
    st = lib().exo_gemm_get_info(handle, ctypes.byref(info))
    if st != OK:
        raise ExoGemmError(st, "exo_gemm_get_info")
    return info


def exo_gemm_destroy(handle) -> int:
    return lib().exo_gemm_destroy(handle)


def exo_gemm_status_string(status: int) -> str:
    return lib().exo_gemm_status_string(status).decode()


def exo_gemm_last_cuda_error() -> int:
    return lib().exo_gemm_last_cuda_error()


def exo_gemm_debug_set(handle, timeout_ms: int, skip_k_block: int) -> int:
    return lib().exo_gemm_debug_set(handle, timeout_ms, skip_k_block)


def exo_gemm_run_static(desc: Desc, a_ptr: int, b_ptr: int, c_ptr: int, alpha: float, beta: float,
                        stream: int = 0, blocking: bool = False):
    """The allocation-free GEMM entry point: no plan, no cudaMalloc (for callers that may not
    allocate device memory).  Returns (status, detail words or None)."""
    if blocking:
        detail = (ctypes.c_uint32 * 8)()
        st = lib().exo_gemm_run_static(ctypes.byref(desc), a_ptr, b_ptr, c_ptr, alpha, beta, stream, detail)
        return st, list(detail)
    return lib().exo_gemm_run_static(ctypes.byref(desc), a_ptr, b_ptr, c_ptr, alpha, beta, stream, None), None


def exo_gemv_run(M: int, N: int, a_ptr: int, lda: int, x_ptr: int, y_ptr: int, alpha: float, beta: float,
                 stream: int = 0) -> int:
    return lib().exo_gemv_run(M, N, a_ptr, lda, x_ptr, y_ptr, alpha, beta, stream)


def exo_gemv_run_colmajor(M: int, N: int, a_ptr: int, lda: int, x_ptr: int, y_ptr: int, alpha: float, beta: float,
                          stream: int = 0) -> int:
    return lib().exo_gemv_run_colmajor(M, N, a_ptr, lda, x_ptr, y_ptr, alpha, beta, stream)


def exo_gemm_schedule_enumerate(tiles_m, tiles_n, band, along_m, num_workers, worker):
    n = lib().exo_gemm_schedule_enumerate(tiles_m, tiles_n, band, along_m, num_workers, worker, None, None, 0)
    if n < 0:
        raise ValueError("bad schedule arguments")
    om = (ctypes.c_int32 * max(n, 1))()
    on = (ctypes.c_int32 * max(n, 1))()
    lib().exo_gemm_schedule_enumerate(tiles_m, tiles_n, band, along_m, num_workers, worker, om, on, n)
    return [(om[i], on[i]) for i in range(n)]


def exo_gemm_schedule_work(tiles, num_workers, tail_workers, num_k_blocks, worker, snap=0, owner_extra=0):
    """[(tile, slice, slices, kb_begin, kb_end), ...] for one worker; the k-blocks of the tail tiles are
    shared among `tail_workers` workers in equal consecutive ranges (0: the tail tiles stay whole)."""
    n = lib().exo_gemm_schedule_work(tiles, num_workers, tail_workers, num_k_blocks, snap, owner_extra, worker,
                                     None, None, None, None, None, 0)
    if n < 0:
        raise ValueError("bad work-schedule arguments")
    t = (ctypes.c_int64 * max(n, 1))()
    s, c, b, e = ((ctypes.c_int32 * max(n, 1))() for _ in range(4))
    lib().exo_gemm_schedule_work(tiles, num_workers, tail_workers, num_k_blocks, snap, owner_extra, worker, t, s, c, b, e, n)
    return [(t[i], s[i], c[i], b[i], e[i]) for i in range(n)]


# ---- thin convenience wrapper ---------------------------------------------------------
class Plan:
    """Owns one handle.  ``run`` takes raw device pointers (ints) and a stream handle."""

    def __init__(self, desc: Desc, batch=None):
        """``batch`` = (count, stride_a, stride_b, stride_c) in elements for a strided batch."""
        if batch is None:
            st, h = exo_gemm_create(desc)
        else:
            st, h = exo_gemm_create_batched(desc, *batch)
        if st != OK:
            raise ExoGemmError(st, "exo_gemm_create")
        self.handle = h
        self.desc = desc

    def run(self, a_ptr, b_ptr, c_ptr, alpha=1.0, beta=0.0, stream=0):
        st = exo_gemm_run(self.handle, a_ptr, b_ptr, c_ptr, alpha, beta, stream)
        if st != OK:
            raise ExoGemmError(st, "exo_gemm_run")

    def check(self):
        st, detail = exo_gemm_check(self.handle)
        if st != OK:
            raise ExoGemmError(st, f"exo_gemm_check {detail}")

    def info(self) -> dict:
        return exo_gemm_get_info(self.handle).as_dict()

    def close(self):
        if self.handle is not None:
            exo_gemm_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
