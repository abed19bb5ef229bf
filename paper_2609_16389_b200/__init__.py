"""B200 (sm_100a) tensor-core GEMM behind a C ABI: C = alpha*A*B + beta*C.

``binding``  ctypes wrappers named after the C entry points (exo_gemm_create / run / destroy ...)
``harness``  device-memory plumbing (PyTorch for memory and streams only)
``synth``    seeded synthetic inputs (shared with the test oracle; no GEMM arithmetic)
``build``    in-tree nvcc build of libexo_gemm.so
"""
__all__ = ["binding", "harness", "synth", "build"]
