"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libexo_gemm.so")
# The same library with the shared-operand cluster kernels compiled in.  Those kernels use a form of TMA
# load that only single-GPU programs may contain, so their source directory and this file are left
# out of multi-GPU deployments, which then run on the base library.
SHARE_DIR = os.path.join(CSRC, "cluster4")
SHARE_LIB = os.path.join(HERE, "libexo_gemm_cluster4.so")
SHARE_DEPS = [os.path.join("cluster4", "share_pairs.cuh")]
SOURCES = ["api.cu", "gemv.cu"]
DEPS = ["api.cu", "gemv.cu", "gemm_kernel.cuh", "gemm_params.h", "plan.h", "ptx.cuh", "tile_scheduler.h",
        os.path.join("..", "..", "include", "exo_gemm.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale(lib: str = LIB, deps=DEPS) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in deps)


def _compile(lib: str, defines, verbose: bool) -> str:
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fno-gnu-unique", "-cudart", "static", "-o", tmp]
    cmd += [f"-D{d}" for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """The base library."""
    if not force and not is_stale():
        return LIB
    return _compile(LIB, [], verbose)


def have_share_sources() -> bool:
    return all(os.path.exists(os.path.join(CSRC, d)) for d in SHARE_DEPS)


def build_share(force: bool = False, verbose: bool = False) -> str:
    """The variant library; raises if its sources are not present."""
    if not have_share_sources():
        raise RuntimeError("the shared-operand cluster sources are not part of this deployment")
    if not force and not is_stale(SHARE_LIB, DEPS + SHARE_DEPS):
        return SHARE_LIB
    return _compile(SHARE_LIB, ["EXO_GEMM_SHARE_PAIRS"], verbose)


def multi_gpu_job() -> bool:
    """True in a process that is one rank of several (torchrun sets WORLD_SIZE)."""
    try:
        return int(os.environ.get("WORLD_SIZE", "1")) > 1
    except ValueError:
        return False


def build_preferred() -> str:
    """The library this process should load: the variant where it can be built and the program runs on
    one GPU, else the base library.  A rank of a multi-GPU job always gets the base library, whatever
    files are present: code that spans several GPUs carries no cluster-multicast load."""
    if os.environ.get("EXO_GEMM_BASE_ONLY") != "1" and not multi_gpu_job() and have_share_sources():
        return build_share()
    return build()


def build_all(force: bool = False, verbose: bool = False):
    """Both libraries (the variant only where its sources are present), compiled side by side."""
    from concurrent.futures import ThreadPoolExecutor
    jobs = [build] + ([build_share] if have_share_sources() else [])
    with ThreadPoolExecutor(len(jobs)) as ex:
        return list(ex.map(lambda fn: fn(force, verbose), jobs))


if __name__ == "__main__":
    print(build_all(force="--force" in sys.argv, verbose="-v" in sys.argv))
