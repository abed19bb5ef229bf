"""The N > 1 benchmark path on CPU: two gloo ranks, each with its own independent
GEMMs (no data-path collective); the job's throughput is all ranks' work divided
by the slowest rank's time."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["EXO_ROOT"])
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
p0 = bench.make_problem("cfg1_256", 0)
pr = bench.make_problem("cfg1_256", rank)
local_ms = 2.0 if rank == 0 else 5.0           # rank 1 is the slow one
tflops, max_ms = bench.aggregate_over_ranks(local_ms, 3.0e12, world)
same_as_rank0 = bool((pr.A == p0.A).all())
# a rank of a multi-GPU job resolves to the base library (no cluster-multicast load in it)
from paper_2609_16389_b200 import binding, build
lib_name = os.path.basename(binding.lib()._name)
has_share = int(binding.exo_gemm_has_shared_operand_clusters())
print("RESULT " + json.dumps({"rank": rank, "tflops": tflops, "max_ms": max_ms, "same_inputs": same_as_rank0,
                              "lib": lib_name, "base": os.path.basename(build.LIB), "has_share": has_share}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_by_slowest_rank():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), EXO_ROOT=ROOT)
        env.pop("EXO_GEMM_LIBRARY", None)
        env.pop("EXO_GEMM_BASE_ONLY", None)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    results = {}
    for pr in procs:
        out, err = pr.communicate(timeout=300)
        assert pr.returncode == 0, err[-2000:]
        line = [l for l in out.splitlines() if l.startswith("RESULT ")][-1]
        r = json.loads(line[len("RESULT "):])
        results[r["rank"]] = r
    for rank in (0, 1):
        assert results[rank]["max_ms"] == 5.0                          # max over ranks, on every rank
        assert abs(results[rank]["tflops"] - (2 * 3.0e12) / 5.0e-3 / 1e12) < 1e-9   # both ranks' work
    assert results[0]["same_inputs"] and not results[1]["same_inputs"]  # independent problems per rank
    for rank in (0, 1):
        assert results[rank]["lib"] == results[rank]["base"] and results[rank]["has_share"] == 0


def test_share_always_is_refused_on_several_gpus():
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    src = ("import sys, types; sys.argv = ['bench.py', '--share', 'always', '--gpus', '2'];"
           "import torch; torch.cuda.is_available = lambda: True;"
           "import bench; bench.main()")
    r = subprocess.run([sys.executable, "-c", src], env=env, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0 and "single-GPU option" in r.stderr, (r.returncode, r.stderr[-1500:])


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    tflops, ms = bench.aggregate_over_ranks(4.0, 8.0e12, 1)
    assert ms == 4.0 and abs(tflops - 2000.0) < 1e-9


def test_reference_arm_prints_one_json_line():
    import json
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--warmup", "1", "--workload", "cfg1_256"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
