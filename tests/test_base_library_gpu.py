"""The base library (libexo_gemm.so) on the GPU.

A single-GPU process loads the variant library, which is the base library plus the shared-operand
cluster kernels; a program that spans several GPUs loads the base library, which contains no
cluster-multicast load at all.  The other GPU tests therefore never map the base library.  This one
runs a child process that is told to load it (EXO_GEMM_BASE_ONLY=1) and checks, against the CPU
oracle: the smoke cases, the 256^3 configuration, a K-sliced tail, a strided batch, a tf32 case and
the allocation-free entry point.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, os.environ["EXO_ROOT"])
import numpy as np
import torch
import oracle
import __graft_entry__ as entry
from paper_2609_16389_b200 import binding as B, build, harness, synth

TOL = 1e-3
assert os.path.basename(B.lib()._name) == os.path.basename(build.LIB), B.lib()._name
assert B.exo_gemm_has_shared_operand_clusters() == 0
# a request for the shared-operand clusters is refused, not silently ignored
d = B.make_desc(512, 512, 256, B.BF16, B.FP32, 0, 1, 0, flags2=B.FLAG2_SHARE_ALWAYS)
assert B.exo_gemm_create(d)[0] == B.ERR_UNSUPPORTED


def check(p, flags=0):
    cbuf, info = harness.gemm_host(p, flags)
    got = oracle.logical_view(cbuf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype)
    cref, den = oracle.gemm_problem(p)
    gate = TOL * den + oracle.output_rounding_slack(cref, p.c_dtype)
    assert (np.abs(got - cref) <= gate).all(), (p.name, info)
    return cbuf, info

for p in entry.smoke_cases():                       # includes the 256^3 configuration
    check(p.generate())
# one whole wave on 8 pairs, then two tail tiles cut along K
p = synth.Problem("base_split", 512, 1280, 4096, synth.FP16, synth.FP32, 0, 1, 0, 1.0, 0.0, seed=5, dist="normal").generate()
_, info = check(p, B.flag_cta_group(2) | B.flag_tile_n(256) | B.flag_grid_limit(16))
assert info["split_k"] >= 2 and info["workspace_bytes"] > 0, info
check(synth.Problem("base_tf32", 264, 328, 200, synth.FP32, synth.FP32, 1, 0, 0, 1.5, 0.5, seed=6).generate())
check(synth.Problem("base_tall", 1024, 512, 264, synth.BF16, synth.BF16, 0, 1, 0, 1.0, 0.0, seed=7).generate())

# strided batch
bp = synth.BatchedProblem("base_batch", 4, 300, 200, 136, synth.BF16, synth.FP32, 0, 1, 0, 1.0, 0.0, seed=8).generate()
dev = torch.device("cuda:0")
dA, dB, dC = (harness._to_device(x, dev) for x in (bp.A, bp.B, bp.C))
with B.Plan(harness.desc_of(bp), batch=(4, bp.stride_a, bp.stride_b, bp.stride_c)) as plan:
    plan.run(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.0, torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize(dev)
    plan.check()
out = dC.cpu().numpy().view(np.float32)
for i in range(4):
    q = bp.matrix(i)
    got = oracle.logical_view(out[i * bp.stride_c:(i + 1) * bp.stride_c], q.M, q.N, 0, q.ldc, synth.FP32)
    assert oracle.max_error(got, *oracle.gemm_problem(q)) <= TOL

# the allocation-free entry point
p = synth.Problem("base_static", 1000, 520, 264, synth.FP16, synth.FP32, 0, 0, 0, 0.5, 1.0, seed=9, dist="normal").generate()
dA, dB, dC = (harness._to_device(x, dev) for x in (p.A, p.B, p.C))
st, detail = B.exo_gemm_run_static(harness.desc_of(p), dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), p.alpha, p.beta,
                                   torch.cuda.current_stream(dev).cuda_stream, blocking=True)
assert st == B.OK and detail[0] == 0, (st, detail)
got = oracle.logical_view(dC.cpu().numpy().view(np.float32), p.M, p.N, 0, p.ldc, synth.FP32)
assert oracle.max_error(got, *oracle.gemm_problem(p)) <= TOL

# fp32 GEMV lives in the base library too
M, N = 300, 1000
rng = np.random.default_rng(3)
A = rng.uniform(-1, 1, M * N).astype(np.float32); x = rng.uniform(-1, 1, N).astype(np.float32); y = np.zeros(M, np.float32)
dA, dx, dy = (harness._to_device(v, dev) for v in (A, x, y))
assert B.exo_gemv_run(M, N, dA.data_ptr(), N, dx.data_ptr(), dy.data_ptr(), 1.0, 0.0) == B.OK
torch.cuda.synchronize(dev)
yref, den = oracle.gemv(M, N, A, N, x, y, 1.0, 0.0)
assert oracle.max_error(dy.cpu().numpy().view(np.float32).astype(np.float64), yref, den) <= TOL
print("BASE_LIBRARY_OK")
"""


def test_base_library_computes_on_the_gpu():
    env = dict(os.environ, EXO_GEMM_BASE_ONLY="1", EXO_ROOT=ROOT)
    env.pop("EXO_GEMM_LIBRARY", None)
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    assert "BASE_LIBRARY_OK" in r.stdout


def test_a_rank_of_a_multi_gpu_job_loads_the_base_library():
    """WORLD_SIZE > 1 in the environment: the binding resolves to the base library whatever files are present."""
    child = ("import os, sys; sys.path.insert(0, os.environ['EXO_ROOT']);"
             "from paper_2609_16389_b200 import binding as B, build;"
             "assert os.path.basename(B.lib()._name) == os.path.basename(build.LIB), B.lib()._name;"
             "assert B.exo_gemm_has_shared_operand_clusters() == 0; print('OK')")
    env = dict(os.environ, WORLD_SIZE="2", EXO_ROOT=ROOT)
    env.pop("EXO_GEMM_LIBRARY", None)
    env.pop("EXO_GEMM_BASE_ONLY", None)
    r = subprocess.run([sys.executable, "-c", child], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "OK" in r.stdout, r.stderr[-2000:]
