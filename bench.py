#!/usr/bin/env python
"""Benchmark of the GEMM hot path: one step = one C = alpha*A*B + beta*C through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints one JSON line (rank 0).  ``value`` is whole-job TFLOP/s (2*M*N*K per GEMM)
with the matrices already resident in HBM; ``e2e`` is the same metric through
the same C-ABI call with host buffers (pinned), host<->device copies inside the
timed region.  With N > 1 (torchrun, one rank per GPU) every rank runs its own
independent GEMMs of the same shape (weak scaling, no collective on the data
path); the time is the maximum over ranks.

``--impl reference`` times the CPU oracle (oracle/) on the host cores, on
bounded row bands of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "GEMM TFLOP/s on 1 B200 and % of dense bf16 tensor-core roofline"
UNIT = "TFLOP/s"
L2_BYTES = 126 * 1024 * 1024

WORKLOADS = {
    # name: (config index, variant)
    "cfg1_256": (0, None), "cfg2_4096": (1, None), "cfg3_8192": (2, None),
    "cfg4a_skinny": (3, "a"), "cfg4b_skinny": (3, "b"),
}
DEFAULT_WORKLOAD = "cfg2_4096"   # the configuration the metric is quoted on; fits one GPU


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--verify", action="store_true",
                    help="sweep only: host-generated inputs for one operand set of every shape and the oracle's "
                         "verdict on 4096 sampled entries per shape (adds several minutes)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the sustained run and the short runs of the other configurations")
    ap.add_argument("--no-cublas", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="EXO_GEMM_FLAG_* overrides (experiments)")
    ap.add_argument("--share", default="auto", choices=["auto", "never", "always"],
                    help="shared-operand 4-CTA clusters (needs the variant library; single-GPU runs only)")
    ap.add_argument("--cta-rows", default="auto", choices=["auto", "128", "256"],
                    help="rows of C per CTA of the 2-CTA tile (256 = the tall tile)")
    return ap.parse_args()


def make_problem(name: str, rank: int = 0):
    from paper_2609_16389_b200 import synth
    if name.startswith("batched_"):
        batch, n = (int(x) for x in name[len("batched_"):].split("x"))
        p = synth.batched(batch, n)
    elif name.startswith("tf32_"):
        p = synth.tf32_square(int(name[len("tf32_"):]))
    elif name.startswith("sweep_"):
        M, N, K = (int(x) for x in name[len("sweep_"):].split("x"))
        p = synth.sweep_problem(M, N, K)
    else:
        idx, variant = WORKLOADS[name]
        p = synth.config(idx, variant)
    p.seed += 7919 * rank      # independent problems per rank
    return p.generate()


def peaks():
    """Measured roofline denominators (generated file), else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "tflops_burst": d["bf16_tflops"],
                "tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


def profiled_traffic(workload: str):
    """DRAM bytes per launch from the committed ncu summary for this workload, if any."""
    path = os.path.join(ROOT, "profiles", f"exo_gemm_kernel_{workload}.md")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        if ln.startswith("dram_bytes_per_launch:"):
            try:
                return float(ln.split(":", 1)[1].split()[0])
            except ValueError:
                return None
    return None


def hold_stream(dev, microseconds):
    """Keeps the current stream of `dev` busy for about that long, so that launches enqueued right after it are
    all queued before the first of them starts: the timed kernels then run back to back on the device
    whatever the host does meanwhile (the clock sampler forks a process every 50 ms)."""
    import torch
    with torch.cuda.device(dev):
        torch.cuda._sleep(int(microseconds * 2000))   # spin cycles; the SM clock is at most 2 GHz


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self._stop = threading.Event()
        self._thr = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                     timeout=5).stdout.strip()
                if out:
                    self.samples.append([x.strip() for x in out.split(",")])
            except Exception:
                pass
            self._stop.wait(0.05)

    def start(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def stop(self, skip_first: int = 0):
        """``skip_first`` drops that many leading samples (taken while the GPU was still ramping up)."""
        self._stop.set()
        if self._thr:
            self._thr.join(timeout=10)
        if skip_first and len(self.samples) > skip_first + 2:
            self.samples = self.samples[skip_first:]
        sm = [float(s[0]) for s in self.samples if s and s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in self.samples if len(s) > 1 and s[1].replace(".", "").isdigit()]
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            for i, n in enumerate(names):
                if len(s) > 3 + i and s[3 + i].lower().startswith("active"):
                    reasons.add(n)
        pw = []
        for smp in self.samples:
            try:
                pw.append(float(smp[2]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w_max": max(pw) if pw else None}


def aggregate_over_ranks(local_ms: float, local_flop: float, world: int, device=None):
    """Whole-job throughput: all ranks' work divided by the slowest rank's time.

    Returns (tflops, max_ms).  Uses one all_reduce(MAX) and one all_reduce(SUM) on
    the default process group when world > 1 (control path only, not data path).
    """
    if world <= 1:
        return local_flop / (local_ms * 1e-3) / 1e12, local_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    f = torch.tensor([local_flop], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(f.item()) / (float(t.item()) * 1e-3) / 1e12, float(t.item())


# ---------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------
def run_reference(args, rank, world):
    if rank != 0:
        return
    import oracle
    p = make_problem(args.workload)
    if getattr(p, "batch", 1) > 1:
        p = p.matrix(0)
    cores = oracle.num_threads()
    # calibrate on a thin band, then size the per-step band so the whole run stays bounded
    cal_rows = min(p.M, 16)
    t0 = time.perf_counter()
    oracle.gemm_problem(p, rows=(0, cal_rows))
    cal = time.perf_counter() - t0
    budget_s = 90.0
    per_row = max(cal / cal_rows, 1e-9)
    rows = int(budget_s / ((args.steps + args.warmup) * per_row))
    rows = max(1, min(p.M, rows))
    for w in range(args.warmup):
        r0 = (w * rows) % max(1, p.M - rows + 1)
        oracle.gemm_problem(p, rows=(r0, r0 + rows))
    t0 = time.perf_counter()
    for s in range(args.steps):
        r0 = ((s + args.warmup) * rows) % max(1, p.M - rows + 1)
        oracle.gemm_problem(p, rows=(r0, r0 + rows))
    dt = time.perf_counter() - t0
    flop = 2.0 * rows * p.N * p.K * args.steps
    tflops = flop / dt / 1e12
    sample = f"each step = a band of {rows} rows of C ({rows}x{p.N}x{p.K}) of {args.workload}"
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": args.workload, "M": p.M, "N": p.N, "K": p.K, "sample": sample},
        "cpu_baseline": {"value": tflops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------
def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2609_16389_b200 import binding as B
    from paper_2609_16389_b200 import harness, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the GEMM path has no CPU fallback")
    if world > 1:
        # several GPUs: the base library only (it holds no cluster-multicast load), whatever files are present
        if args.share == "always":
            raise SystemExit("bench.py: --share always is a single-GPU option (the shared-operand clusters "
                             "are not part of a multi-GPU program)")
        os.environ["EXO_GEMM_BASE_ONLY"] = "1"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    p = make_problem(args.workload, rank)
    flop = p.flop
    set_bytes = p.A.nbytes + p.B.nbytes + p.C.nbytes
    n_sets = max(2, int(np.ceil(2.0 * L2_BYTES / set_bytes)))     # rotate through > 2x L2 of operands
    n_sets = min(n_sets, 64)
    sets = []
    for _ in range(n_sets):
        sets.append((harness._to_device(p.A, dev), harness._to_device(p.B, dev), harness._to_device(p.C, dev)))
    batch = getattr(p, "batch", 1)
    flags2 = {"auto": B.FLAG2_SHARE_AUTO, "never": B.FLAG2_SHARE_NEVER, "always": B.FLAG2_SHARE_ALWAYS}[args.share]
    if args.cta_rows != "auto":
        flags2 |= B.flag2_cta_rows(int(args.cta_rows))
    plan = B.Plan(harness.desc_of(p, args.flags, local_rank, flags2),
                  batch=(batch, p.stride_a, p.stride_b, p.stride_c) if batch > 1 else None)
    info = plan.info()
    stream = torch.cuda.current_stream(dev)

    def step(i):
        a, b, c = sets[i % n_sets]
        plan.run(a.data_ptr(), b.data_ptr(), c.data_ptr(), p.alpha, p.beta, stream.cuda_stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    # --- device-resident timing: exactly K steps, back to back, bracketed by two events on the launching
    # stream (an event between every two launches costs each step 2-4 % of a 96 us kernel: it keeps the next
    # kernel's programmatic early start from overlapping the previous one's tail)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    hold_stream(dev, 8.0 * args.steps + 50.0)   # the host enqueues the K steps while the stream is held
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
    ev1.record(stream)
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    plan.check()
    # per-step spread, from a second, untimed pass with an event after every step
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record(stream)
    for i in range(args.steps):
        step(i)
        ev[i + 1].record(stream)
    barrier()
    per_step = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)])
    plan.check()

    # --- cuBLAS on the same box, same shapes (reference point only), interleaved order
    cublas = None
    if rank == 0 and not args.no_cublas:
        cublas = time_cublas(p, dev, args.steps, n_sets, ours_step=step)

    # --- end to end: pinned host buffers, H2D + GEMM + D2H inside the timed region
    e2e_steps = max(3, min(args.steps, 20))
    e2e = end_to_end(p, dev, stream, plan, sets[0], e2e_steps, barrier, args.flags, flags2, local_rank)
    e2e_ms, h2d, d2h = e2e["ms_per_step"], e2e["h2d_bytes_per_step"], e2e["d2h_bytes_per_step"]
    clocks = sampler.stop()
    plan.check()

    # --- sustained: the same back-to-back launches for about a second of device time, with clock samples
    # taken inside that region only (the K-step region above is over before the sampler's second reading)
    sustained = None
    if world == 1 and not args.no_extras:
        n_long = int(min(200000, max(args.steps, np.ceil(1000.0 / max(total_ms / args.steps, 1e-3)))))
        long_sampler = ClockSampler(local_rank)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        s0.record(stream)
        long_sampler.start()
        for i in range(n_long):
            step(i)
        s1.record(stream)
        barrier()
        long_clocks = long_sampler.stop(skip_first=2)
        plan.check()
        long_ms = s0.elapsed_time(s1)
        sustained = {"tflops": flop * n_long / (long_ms * 1e-3) / 1e12, "steps": n_long, "seconds": long_ms * 1e-3,
                     "clocks": long_clocks}

    value, max_ms = aggregate_over_ranks(total_ms, flop * args.steps, world, dev)
    e2e_value, _ = aggregate_over_ranks(e2e_ms, flop, world, dev)

    if rank == 0:
        pk = peaks()
        ms_per_step = max_ms / args.steps
        avg_kernel_ms = total_ms / args.steps          # one kernel per step, back to back
        achieved = flop / (avg_kernel_ms * 1e-3) / 1e12
        timed_region_s = total_ms * 1e-3
        peak = pk["tflops_burst"] if timed_region_s < 1.0 else pk["tflops_sustained"]
        if p.ab_dtype == synth.FP32:   # tf32: the bf16 measurement times the nominal tf32/bf16 ratio (1.1 / 2.25)
            peak *= 1.1 / 2.25
        ai = flop / p.algorithmic_bytes
        hbm_bound_tflops = ai * pk["hbm_gbs"] / 1e3
        tensor_bound = hbm_bound_tflops >= peak
        q1, q3 = np.percentile(per_step, [25, 75])
        iqr = per_step[(per_step >= q1) & (per_step <= q3)]
        roofline = {
            "bound": "tensor" if tensor_bound else "hbm",
            "achieved": achieved if tensor_bound else p.algorithmic_bytes / (avg_kernel_ms * 1e-3) / 1e9,
            "peak": peak if tensor_bound else pk["hbm_gbs"],
            "unit": "TFLOP/s" if tensor_bound else "GB/s",
            "traffic": profiled_traffic(args.workload),
            "peak_source": f"{pk['source']} ({'burst' if timed_region_s < 1.0 else 'sustained'} cuBLAS bf16)"
                           if tensor_bound else f"{pk['source']} (copy bandwidth)",
            "kernel": (f"exo_gemm_lean_kernel<{info['tile_n']}>" if info.get('lean_kernel') else f"exo_gemm_kernel<{info['cta_group']},{info['tile_n']}>"),
            "avg_kernel_ms": avg_kernel_ms,
            "algorithmic_bytes": p.algorithmic_bytes, "flop": flop,
            "frac_of_nominal_2250": achieved / 2250.0,
        }
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": {synth.BF16: "bf16", synth.FP16: "fp16", synth.FP32: "tf32"}[p.ab_dtype] + " in, fp32 accumulate",
            "data": "synthetic",
            "config": {"workload": args.workload, "M": p.M, "N": p.N, "K": p.K, "batch": batch,
                       "ab_dtype": synth.dtype_name(p.ab_dtype), "c_dtype": synth.dtype_name(p.c_dtype),
                       "layouts": "A%s B%s C%s" % tuple("rc"[x] for x in (p.a_layout, p.b_layout, p.c_layout)),
                       "alpha": p.alpha, "beta": p.beta,
                       "l2": f"rotating {n_sets} operand sets ({n_sets * set_bytes >> 20} MiB > 126 MiB L2)",
                       "timing": "two CUDA events around the K steps on the launching stream; the stream is held by a spin "
                                 "kernel in front of the first event while the host enqueues the steps",
                       "plan": info},
            "iqr_mean_ms": float(iqr.mean()) if iqr.size else None, "min_ms": float(per_step.min()),
            "roofline": roofline,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "how": e2e["how"], "parity": e2e["parity"]},
            "gpu_launches": args.steps,
            "clocks": clocks,
        }
        if cublas is not None:
            line["cublas"] = cublas
        if sustained is not None:
            speak = pk["tflops_sustained"] * (1.1 / 2.25 if p.ab_dtype == synth.FP32 else 1.0)
            sustained["peak"] = speak
            sustained["frac"] = sustained["tflops"] / speak
            sustained["peak_source"] = f"{pk['source']} (sustained cuBLAS bf16)"
            line["sustained"] = sustained
        if world == 1 and not args.no_extras and args.workload == DEFAULT_WORKLOAD:
            # the other benchmark configurations, a short run each (their own bench lines: --workload NAME)
            line["configs"] = {}
            for name in ("cfg1_256", "cfg3_8192", "cfg4a_skinny", "cfg4b_skinny"):
                try:
                    line["configs"][name] = measure_config(name, dev, max(3, min(args.steps, 20)), pk)
                except Exception as e:   # a side measurement never fails the headline
                    line["configs"][name] = {"error": repr(e)}
            line["configs"][args.workload] = {"M": p.M, "N": p.N, "K": p.K, "tflops": value, "frac": roofline["frac"],
                                              "parity": sampled_parity(p, sets[(args.steps - 1) % n_sets][2].cpu().numpy()
                                                                       .view(synth.storage_np_dtype(p.c_dtype)))
                                              if p.beta == 0.0 else None}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(p, args.workload)
        print(json.dumps(line), flush=True)

    plan.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def sampled_parity(p, cbuf, n=1 << 14):
    """Oracle error metric of a finished GEMM on n random entries of C (the oracle computes them one by one)."""
    import oracle
    rng = np.random.default_rng(p.seed)
    r, c = rng.integers(0, p.M, n), rng.integers(0, p.N, n)
    got = oracle.logical_view(cbuf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype)[r, c]
    cref, den = oracle.gemm_problem_entries(p, r, c)
    return {"max_error_metric": oracle.max_error(got, cref, den), "tolerance": oracle.TOLERANCE, "entries": int(n)}


def measure_config(name, dev, steps, pk):
    """A short run of one benchmark configuration: TFLOP/s over `steps` launches back to back (operand sets
    rotated past L2), roofline fraction, the plan, and the oracle's verdict on sampled entries."""
    import torch
    from paper_2609_16389_b200 import binding as B
    from paper_2609_16389_b200 import harness, synth
    p = make_problem(name)
    set_bytes = p.A.nbytes + p.B.nbytes + p.C.nbytes
    n_sets = int(min(8, max(2, np.ceil(2.0 * L2_BYTES / set_bytes))))
    sets = [(harness._to_device(p.A, dev), harness._to_device(p.B, dev), harness._to_device(p.C, dev)) for _ in range(n_sets)]
    stream = torch.cuda.current_stream(dev)
    with B.Plan(harness.desc_of(p, 0, dev.index or 0)) as plan:
        info = plan.info()

        def step(i):
            a, b, c = sets[i % n_sets]
            plan.run(a.data_ptr(), b.data_ptr(), c.data_ptr(), p.alpha, p.beta, stream.cuda_stream)

        # parity first, on a fresh C (beta != 0 updates C in place, so later steps change it again)
        step(0)
        torch.cuda.synchronize(dev)
        plan.check()
        parity = sampled_parity(p, sets[0][2].cpu().numpy().view(synth.storage_np_dtype(p.c_dtype)))
        for i in range(3):
            step(i)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        hold_stream(dev, 8.0 * steps + 50.0)
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        plan.check()
        ms = e0.elapsed_time(e1) / steps
        graph_ms = None
        if ms < 0.02 and p.beta == 0.0:
            # A step this short is bounded by the host's launch path (three tensor maps and a launch per call):
            # the same launches captured into a CUDA graph and replayed give the kernels back to back.
            side = torch.cuda.Stream(dev)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(steps):
                    a, b, c = sets[i % n_sets]
                    plan.run(a.data_ptr(), b.data_ptr(), c.data_ptr(), p.alpha, p.beta, side.cuda_stream)
            graph.replay()
            torch.cuda.synchronize(dev)
            e0.record(stream)
            for _ in range(10):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize(dev)
            plan.check()
            graph_ms = e0.elapsed_time(e1) / (10 * steps)
            del graph
    tf = p.flop / (ms * 1e-3) / 1e12
    roof = min(pk["tflops_burst"], p.flop / p.algorithmic_bytes * pk["hbm_gbs"] / 1e3)
    extra = {} if graph_ms is None else {"graph_replay_ms_per_step": graph_ms, "graph_replay_tflops": p.flop / (graph_ms * 1e-3) / 1e12}
    return {**extra, "M": p.M, "N": p.N, "K": p.K, "tflops": tf, "ms_per_step": ms, "steps": steps,
            "roofline_tflops": roof, "frac": tf / roof,
            "hbm_gbs": p.algorithmic_bytes / (ms * 1e-3) / 1e9,
            "plan": {k: info[k] for k in ("cta_group", "tile_m", "tile_n", "tile_k", "stages", "epilogue_buffers",
                                          "split_k", "tail_tiles", "grid", "lean_kernel")},
            "l2_sets": n_sets, "parity": parity}


def end_to_end(p, dev, stream, plan, dev_set, steps, barrier, flags, flags2, local_rank):
    """The same GEMM with HOST buffers: every step uploads its A, B (and C_in if beta != 0) from pinned host
    memory, computes through exo_gemm_run, and reads its C back to pinned host memory, all inside the
    timed region.

    Where A and C are row-major the step is pipelined over row bands of C: one stream uploads B and then A
    band by band, the compute stream runs one exo_gemm_run per band (a plan over a band, base pointers
    offset) as soon as that band and B have landed, a third stream downloads each finished band of C.
    PCIe carries both directions at once, and with two sets of device buffers the next step's upload
    overlaps this step's download.  Otherwise: upload, one GEMM, download, on one stream.
    """
    import torch
    from paper_2609_16389_b200 import binding as B
    from paper_2609_16389_b200 import harness, synth
    batch = getattr(p, "batch", 1)
    hA = torch.from_numpy(p.A.view(np.uint8)).pin_memory()
    hB = torch.from_numpy(p.B.view(np.uint8)).pin_memory()
    hC = torch.from_numpy(p.C.view(np.uint8)).pin_memory()
    hOut = torch.empty_like(hC).pin_memory()
    need_c_in = p.beta != 0.0
    h2d = hA.numel() + hB.numel() + (hC.numel() if need_c_in else 0)
    d2h = hOut.numel()
    bands = 0
    if batch == 1 and p.a_layout == synth.ROW_MAJOR and p.c_layout == synth.ROW_MAJOR and p.M >= 2048:
        for nb in (8, 4, 2):
            if p.M % (nb * 256) == 0:
                bands = nb
                break

    if not bands:
        dA, dB, dC = dev_set

        def step():
            dA.copy_(hA, non_blocking=True)
            dB.copy_(hB, non_blocking=True)
            if need_c_in:
                dC.copy_(hC, non_blocking=True)
            plan.run(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), p.alpha, p.beta, stream.cuda_stream)
            hOut.copy_(dC, non_blocking=True)

        for _ in range(2):
            step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1) / steps
        how = "serial: H2D, one exo_gemm_run, D2H on one stream"
    else:
        rows = p.M // bands
        es_ab, es_c = synth.elem_size(p.ab_dtype), synth.elem_size(p.c_dtype)
        a_band, c_band = rows * p.lda * es_ab, rows * p.ldc * es_c      # bytes per band (row-major, rows apart by ld)
        band_desc = B.make_desc(rows, p.N, p.K, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout, p.c_layout,
                                p.lda, p.ldb, p.ldc, device=local_rank, flags=flags, flags2=flags2)
        band_plan = B.Plan(band_desc)
        dsets = [tuple(torch.empty_like(t) for t in dev_set) for _ in range(2)]
        up, down = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        busy = [None, None]     # last event of the step that used a device set (its download), before the set is reused

        def step(k):
            dA, dB, dC = dsets[k % 2]
            with torch.cuda.stream(up):
                if busy[k % 2] is not None:
                    up.wait_event(busy[k % 2])
                dB.copy_(hB, non_blocking=True)
                landed = []
                for i in range(bands):
                    dA[i * a_band:(i + 1) * a_band].copy_(hA[i * a_band:(i + 1) * a_band], non_blocking=True)
                    if need_c_in:
                        dC[i * c_band:(i + 1) * c_band].copy_(hC[i * c_band:(i + 1) * c_band], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(up)
                    landed.append(ev)
            for i in range(bands):
                stream.wait_event(landed[i])
                band_plan.run(dA.data_ptr() + i * a_band, dB.data_ptr(), dC.data_ptr() + i * c_band, p.alpha, p.beta,
                              stream.cuda_stream)
                done = torch.cuda.Event()
                done.record(stream)
                with torch.cuda.stream(down):
                    down.wait_event(done)
                    hOut[i * c_band:(i + 1) * c_band].copy_(dC[i * c_band:(i + 1) * c_band], non_blocking=True)
            last = torch.cuda.Event()
            last.record(down)
            busy[k % 2] = last
            return last

        for k in range(2):
            step(k)
        barrier()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        up.wait_stream(stream)
        e0.record(up)
        stream.wait_event(e0)
        last = None
        for k in range(steps):
            last = step(k)
        stream.wait_event(last)          # the step's result is on the host when the timed region ends
        e1.record(stream)
        barrier()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / steps
        band_plan.check()
        band_plan.close()
        how = (f"pipelined over {bands} row bands of C: upload stream (B, then A band by band), one exo_gemm_run per band, "
               "download stream; two device buffer sets")
    parity = None
    if batch == 1:
        parity = sampled_parity(p, hOut.numpy().view(synth.storage_np_dtype(p.c_dtype)), 1 << 12)
    return {"ms_per_step": ms, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "how": how, "parity": parity}


def time_cublas(p, dev, steps, n_sets, ours_step=None):
    """torch.matmul / addmm (cuBLAS) on the same shapes: a same-box reference point."""
    import torch
    from paper_2609_16389_b200 import synth
    try:
        tdt = {synth.BF16: torch.bfloat16, synth.FP16: torch.float16, synth.FP32: torch.float32}[p.ab_dtype]
        prev_tf32 = torch.backends.cuda.matmul.allow_tf32
        if p.ab_dtype == synth.FP32:
            torch.backends.cuda.matmul.allow_tf32 = True     # cuBLAS in tf32 tensor-op mode, as in the paper
        batch = getattr(p, "batch", 1)
        if batch > 1:
            a = torch.randn(batch, p.M, p.K, device=dev).to(tdt)
            b = torch.randn(batch, p.N, p.K, device=dev).to(tdt).transpose(1, 2)
            c = torch.empty(batch, p.M, p.N, device=dev, dtype=tdt)
            for _ in range(3):
                torch.bmm(a, b, out=c)
            torch.cuda.synchronize(dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                torch.bmm(a, b, out=c)
            e1.record()
            torch.cuda.synchronize(dev)
            ms = e0.elapsed_time(e1) / steps
            return {"tflops": p.flop / (ms * 1e-3) / 1e12, "ms_per_step": ms, "note": "torch.bmm, same shapes (L2-warm)"}
        # the same operand values as our arm (tensor-core power, and with it the clock, depends on the data)
        def view(buf, rows, cols, layout, ld):
            t = torch.from_numpy(buf.view(np.int16) if buf.dtype == np.uint16 else buf).to(dev).view(tdt)
            return torch.as_strided(t, (rows, cols), (ld, 1) if layout == synth.ROW_MAJOR else (1, ld))
        sets = []
        for _ in range(n_sets):
            sets.append((view(p.A, p.M, p.K, p.a_layout, p.lda), view(p.B, p.K, p.N, p.b_layout, p.ldb),
                         torch.empty(p.M, p.N, device=dev, dtype=tdt)))
        for i in range(3):
            a, b, c = sets[i % n_sets]
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize(dev)

        def theirs(i):
            a, b, c = sets[i % n_sets]
            torch.matmul(a, b, out=c)

        # The two kernels take turns in blocks, in random order within each round, and each side reports
        # the mean of its inter-quartile range (the protocol of the paper's Section 6).  A GPU at its
        # power cap clocks by its recent history, so timing one side after the other favours whichever
        # runs on the cooler device.
        import random
        rnd = random.Random(0)
        block = max(1, steps // 5)
        rounds = 10
        sides = {"cublas": theirs}
        if ours_step is not None:
            sides["ours"] = ours_step
        ms = {k: [] for k in sides}
        for _ in range(rounds):
            order = list(sides.items())
            rnd.shuffle(order)
            for name, fn in order:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(block):
                    fn(i)
                e1.record()
                torch.cuda.synchronize(dev)
                ms[name].append(e0.elapsed_time(e1) / block)

        def iqr_mean(v):
            v = np.sort(np.array(v))
            q = len(v) // 4
            return float(v[q:len(v) - q].mean())

        out = {"tflops": p.flop / (iqr_mean(ms["cublas"]) * 1e-3) / 1e12, "ms_per_step": iqr_mean(ms["cublas"]),
               "note": "torch.matmul, 16-bit output, alpha=1 beta=0, same M,N,K, operand layouts and operand values; "
                       f"{rounds} rounds of {block}-launch blocks alternating with our kernel in random order, IQR mean"}
        if "ours" in ms:
            out["ours_same_protocol_tflops"] = p.flop / (iqr_mean(ms["ours"]) * 1e-3) / 1e12
        return out
    except Exception as e:  # a reference point only; never fails the bench
        return {"error": repr(e)}


def cpu_baseline(p, workload):
    import oracle
    if getattr(p, "batch", 1) > 1:
        p = p.matrix(0)
    cores = oracle.num_threads()
    cal_rows = min(p.M, 16)
    t0 = time.perf_counter()
    oracle.gemm_problem(p, rows=(0, cal_rows))
    cal = time.perf_counter() - t0
    target_wall = 20.0 / max(cores, 1)       # about 20 s of CPU work in total
    rows = int(max(1, min(p.M, target_wall / max(cal / cal_rows, 1e-9))))
    t0 = time.perf_counter()
    oracle.gemm_problem(p, rows=(0, rows))
    dt = time.perf_counter() - t0
    return {"value": 2.0 * rows * p.N * p.K / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"rows 0..{rows} of C ({rows}x{p.N}x{p.K}) of {workload}, {dt:.1f} s wall"}


def run_sweep(args, rank, world, local_rank):
    """The shape sweep: M, N, K each in {512, 1000, 2048, 3072, 6144, 12288}, bf16 in, fp32 out.

    Operands are drawn on the device, uniform[-1, 1) rounded to bf16 (with --verify one operand set per
    shape is the seeded host-generated problem and its result is checked by the oracle on sampled
    entries; otherwise parity of the sweep is what the GPU tests cover, one shape per plan class).  Every
    shape gets its own plan, 3 warm-up launches and `--steps` launches replayed from a CUDA graph; the
    line reports whole-sweep throughput and, per shape, TFLOP/s and the fraction of
    roofline(shape) = min(tensor peak, AI x HBM bandwidth).
    """
    import itertools
    import torch
    from paper_2609_16389_b200 import binding as B
    from paper_2609_16389_b200 import synth
    if rank != 0:
        return
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pk = peaks()
    stream = torch.cuda.current_stream(dev)
    steps = max(3, min(args.steps, 20))
    side = torch.cuda.Stream(dev)
    rows, tot_flop, tot_ms, launches = [], 0.0, 0.0, 0
    sampler = ClockSampler(local_rank)
    sampler.start()
    from paper_2609_16389_b200 import harness
    worst_parity = 0.0
    for (M, N, K) in itertools.product(synth.SWEEP_DIMS, repeat=3):
        set_bytes = 2 * (M * K + K * N) + 4 * M * N
        n_sets = int(min(8, max(1, np.ceil(2.0 * L2_BYTES / set_bytes))))
        sets = [((torch.rand(M, K, device=dev) * 2 - 1).to(torch.bfloat16),
                 (torch.rand(N, K, device=dev) * 2 - 1).to(torch.bfloat16),
                 torch.empty(M, N, device=dev, dtype=torch.float32)) for _ in range(n_sets)]
        prob = None
        if args.verify:     # operand set 0 holds the seeded host-generated problem of this shape
            prob = synth.sweep_problem(M, N, K).generate()
            sets[0] = (harness._to_device(prob.A, dev), harness._to_device(prob.B, dev), harness._to_device(prob.C, dev))
        plan = B.Plan(B.make_desc(M, N, K, B.BF16, B.FP32, B.ROW_MAJOR, B.COL_MAJOR, B.ROW_MAJOR,
                                  device=local_rank, flags=args.flags))

        def step(i, s=None):
            a, b, c = sets[i % n_sets]
            plan.run(a.data_ptr(), b.data_ptr(), c.data_ptr(), 1.0, 0.0, (s or stream).cuda_stream)

        for i in range(3):
            step(i)
        torch.cuda.synchronize(dev)
        # `steps` launches captured into one CUDA graph and replayed: what is timed is the kernels back to back,
        # not the host's launch rate (which would bound every shape under ~10 us)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(steps):
                step(i, side)
        graph.replay()
        torch.cuda.synchronize(dev)
        reps = 3 if 2.0 * M * N * K > 1e11 else 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        plan.check()
        ms = e0.elapsed_time(e1) / (steps * reps)
        info = plan.info()
        flop = 2.0 * M * N * K
        ai = flop / set_bytes
        roof = min(pk["tflops_burst"], ai * pk["hbm_gbs"] / 1e3)
        tf = flop / (ms * 1e-3) / 1e12
        row = {"M": M, "N": N, "K": K, "us": round(ms * 1e3, 2), "tflops": round(tf, 1),
               "roofline_tflops": round(roof, 1), "frac": round(tf / roof, 3),
               "plan": [info["cta_group"], info["tile_m"], info["tile_n"], info["tile_k"], info["split_k"], info["cluster_size"], info["lean_kernel"]],
               "l2_sets": n_sets}
        if prob is not None:
            step(0)
            torch.cuda.synchronize(dev)
            plan.check()
            par = sampled_parity(prob, sets[0][2].cpu().numpy().view(np.float32), 1 << 12)
            row["parity"] = float("%.3g" % par["max_error_metric"])
            worst_parity = max(worst_parity, par["max_error_metric"])
        plan.close()
        rows.append(row)
        tot_flop += flop * steps
        tot_ms += ms * steps
        launches += steps * (reps + 1) + 3
        del sets, graph
    clocks = sampler.stop()
    fr = np.array([r["frac"] for r in rows])
    line = {
        "metric": METRIC, "value": tot_flop / (tot_ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": 3, "ms_per_step": tot_ms / launches, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in, fp32 accumulate",
        "data": "synthetic (device-generated for timing" + ("; operand set 0 of every shape seeded on the host and checked by the oracle)" if args.verify else ")"),
        "config": {"workload": "sweep_216", "shapes": len(rows), "dims": list(synth.SWEEP_DIMS),
                   "layouts": "Ar Bc Cr", "c_dtype": "fp32",
                   "l2": "operand sets rotated to exceed 2x L2 where 8 sets suffice, else L2-warm (l2_sets per shape)",
                   "timing": f"{steps} launches per shape captured into a CUDA graph, the graph replayed 3 or 10 times between two events",
                   "parity": ({"entries_per_shape": 4096, "worst_max_error_metric": worst_parity, "tolerance": 1e-3}
                              if args.verify else "per plan class in tests/test_gemm_gpu.py; per shape with --verify")},
        "roofline": {"bound": "mixed", "achieved": float(np.exp(np.log(fr).mean())), "peak": 1.0, "unit": "fraction",
                     "frac": float(np.exp(np.log(fr).mean())), "traffic": None,
                     "note": "geometric mean over shapes of TFLOP/s / min(measured tensor peak, AI x measured HBM GB/s)",
                     "min_frac": float(fr.min()), "max_frac": float(fr.max())},
        "gpu_launches": launches, "clocks": clocks, "sweep": rows,
    }
    print(json.dumps(line), flush=True)


def run_gemv(args, rank, world, local_rank):
    """fp32 GEMV y = A x, the paper's memory-bound companion workload (Section 6).
    Workload name gemv_<M>x<N> (row-major A) or gemvc_<M>x<N> (column-major A).  A step = one exo_gemv_run[_colmajor]; the matrices rotate through several copies
    so that every step streams A from HBM.  Roofline: HBM (algorithmic bytes = 4*M*N + 4*N + 4*M)."""
    import torch
    from paper_2609_16389_b200 import binding as B
    if rank != 0:
        return
    col = args.workload.startswith("gemvc_")
    M, N = (int(v) for v in args.workload.split("_", 1)[1].split("x"))
    lda = M if col else N
    run = B.exo_gemv_run_colmajor if col else B.exo_gemv_run
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pk = peaks()
    rng = np.random.default_rng(260916389 + 70)
    hA = rng.uniform(-1, 1, size=M * N).astype(np.float32)
    hx = rng.uniform(-1, 1, size=N).astype(np.float32)
    n_sets = int(max(2, min(16, np.ceil(2.0 * L2_BYTES / hA.nbytes))))
    dAs = [torch.from_numpy(hA).to(dev) for _ in range(n_sets)]
    dx = torch.from_numpy(hx).to(dev)
    dy = torch.zeros(M, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step(i):
        st = run(M, N, dAs[i % n_sets].data_ptr(), lda, dx.data_ptr(), dy.data_ptr(), 1.0, 0.0, stream.cuda_stream)
        if st != B.OK:
            raise B.ExoGemmError(st, "exo_gemv_run")

    for i in range(max(3, args.warmup)):
        step(i)
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / args.steps
    # end to end: A, x from pinned host memory, y back
    pA, px = torch.from_numpy(hA).pin_memory(), torch.from_numpy(hx).pin_memory()
    py = torch.empty(M, dtype=torch.float32).pin_memory()
    k = max(3, min(10, args.steps))
    torch.cuda.synchronize(dev)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for _ in range(k):
        dAs[0].copy_(pA, non_blocking=True)
        dx.copy_(px, non_blocking=True)
        step(0)
        py.copy_(dy, non_blocking=True)
    f1.record(stream)
    torch.cuda.synchronize(dev)
    e2e_ms = f0.elapsed_time(f1) / k
    clocks = sampler.stop()
    flop = 2.0 * M * N
    abytes = 4.0 * (M * N + N + M)
    gbs = abytes / (ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": flop / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "M": M, "N": N, "layout": "A column-major" if col else "A row-major",
                   "l2": f"rotating {n_sets} copies of A ({n_sets * hA.nbytes >> 20} MiB > 126 MiB L2)"},
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                     "traffic": None, "peak_source": f"{pk['source']} (copy bandwidth)", "kernel": "exo_gemv_colmajor_kernel" if col else "exo_gemv_rowmajor_kernel",
                     "algorithmic_bytes": abytes, "flop": flop},
        "e2e": {"value": flop / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": int(hA.nbytes + hx.nbytes),
                "d2h_bytes_per_step": int(4 * M), "ms_per_step": e2e_ms, "steps": k},
        "gpu_launches": args.steps, "clocks": clocks,
    }
    if not args.no_cublas:
        xs = dx
        mat = (lambda t: t.view(N, M).t()) if col else (lambda t: t.view(M, N))
        for _ in range(3):
            torch.mv(mat(dAs[0]), xs, out=dy)
        torch.cuda.synchronize(dev)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for i in range(args.steps):
            torch.mv(mat(dAs[i % n_sets]), xs, out=dy)
        g1.record(stream)
        torch.cuda.synchronize(dev)
        cms = g0.elapsed_time(g1) / args.steps
        line["cublas"] = {"gbs": abytes / (cms * 1e-3) / 1e9, "ms_per_step": cms, "note": "torch.mv (cublasSgemv)"}
    if not args.no_cpu_baseline:
        import oracle
        rows = min(M, max(1, int(2e9 / max(N, 1))))
        t0 = time.perf_counter()
        oracle.gemv(rows, N, hA, lda, hx, np.zeros(rows, np.float32), 1.0, 0.0, layout=1 if col else 0)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 2.0 * rows * N / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
                                "kind": "oracle", "sample": f"rows 0..{rows} of {args.workload}, {dt:.2f} s wall"}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.workload.startswith(("gemv_", "gemvc_")):
        if args.impl == "reference":
            raise SystemExit("the reference arm times GEMM workloads")
        run_gemv(args, rank, world, local_rank)
        return
    if args.workload == "sweep":
        if args.impl == "reference":
            raise SystemExit("the reference arm times one workload; pick e.g. --workload sweep_1000x1000x1000")
        run_sweep(args, rank, world, local_rank)
        return
    if args.workload not in WORKLOADS and not args.workload.startswith(("sweep_", "batched_", "tf32_", "gemv_", "gemvc_")):
        raise SystemExit(f"unknown workload {args.workload}")
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
