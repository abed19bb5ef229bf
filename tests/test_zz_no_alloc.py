"""The allocation-free entry point (exo_gemm_run_static) against the plan-based one.

Some callers of this library cannot allocate device memory when they need a GEMM: all of
the GPU's memory may already belong to a framework's pool, or the call sits in a loop that
must not touch the allocator.  For them the library keeps the kernel's 32-byte status block
in a device array inside the library image instead of a cudaMalloc'ed block.  This test
calls that entry point through the C ABI twice in a row and checks both results against
exo_gemm_create + exo_gemm_run on the same inputs, with the tolerance of the parity tests
(1e-3 of the oracle's denominator; the two paths run the same kernel, so the results are
expected to be identical).  The file name makes pytest collect it last.
"""
import numpy as np
import pytest

import oracle
from paper_2609_16389_b200 import binding as B
from paper_2609_16389_b200 import harness, synth

pytestmark = pytest.mark.gpu
TOL = 1e-3

CASES = [
    synth.Problem("static_fp16_beta", 1000, 520, 264, synth.FP16, synth.FP32, synth.ROW_MAJOR,
                  synth.ROW_MAJOR, synth.ROW_MAJOR, 0.5, 1.0, seed=21, dist="normal"),
    synth.Problem("static_bf16_colmajor_c", 384, 648, 1000, synth.BF16, synth.BF16, synth.COL_MAJOR,
                  synth.COL_MAJOR, synth.COL_MAJOR, 1.0, 0.0, seed=22),
]


@pytest.mark.parametrize("p", CASES, ids=lambda p: p.name)
def test_static_entry_point_matches_the_plan_based_one_twice_in_a_row(p):
    import torch
    p.generate()
    # exo_gemm_create + exo_gemm_run.  K-slicing of tail tiles needs a device workspace, which the
    # allocation-free entry point never uses, so the reference plan is told not to slice either:
    # then both run the same kernel with the same work list.
    want_buf, _ = harness.gemm_host(p, B.flag_split_k(1))
    want = oracle.logical_view(want_buf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype)
    cref, den = oracle.gemm_problem(p)
    slack = oracle.output_rounding_slack(cref, p.c_dtype)
    assert (np.abs(want - cref) <= TOL * den + slack).all()  # the plan-based path itself is right

    dev = torch.device("cuda:0")
    dA, dB = harness._to_device(p.A, dev), harness._to_device(p.B, dev)
    dC1, dC2 = harness._to_device(p.C, dev), harness._to_device(p.C, dev)
    desc = harness.desc_of(p)
    stream = torch.cuda.current_stream(dev).cuda_stream
    # two calls in a row on one stream: the first asynchronous, the second in blocking mode
    st, _ = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC1.data_ptr(), p.alpha, p.beta, stream)
    assert st == B.OK, B.exo_gemm_status_string(st)
    st, detail = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC2.data_ptr(), p.alpha, p.beta,
                                       stream, blocking=True)
    assert st == B.OK and detail[0] == 0, (B.exo_gemm_status_string(st), detail)
    torch.cuda.synchronize(dev)
    for dC in (dC1, dC2):
        buf = dC.cpu().numpy().view(synth.storage_np_dtype(p.c_dtype))
        got = oracle.logical_view(buf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype)
        assert oracle.max_error(got, want, den) <= TOL       # against the existing entry point
        assert np.array_equal(buf, want_buf)                 # same kernel, same work list: same bits
    # and against the library's default plan for this problem (which may slice K), within tolerance
    auto_buf, _ = harness.gemm_host(p)
    auto = oracle.logical_view(auto_buf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype)
    assert (np.abs(got - auto) <= TOL * den + 2 * slack).all()


def test_static_entry_point_checks_its_arguments_like_the_others():
    import torch
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda:0")
    ptr = buf.data_ptr()
    bad = B.make_desc(64, 64, 100, synth.BF16, synth.FP32, 0, 1, 0)          # lda*2 not a multiple of 16
    assert B.exo_gemm_run_static(bad, ptr, ptr, ptr, 1.0, 0.0)[0] == B.ERR_UNSUPPORTED
    ok = B.make_desc(64, 64, 64, synth.BF16, synth.FP32, 0, 1, 0)
    assert B.exo_gemm_run_static(ok, ptr + 2, ptr, ptr + 32768, 1.0, 0.0)[0] == B.ERR_ALIGNMENT
    assert B.exo_gemm_run_static(ok, 0, ptr, ptr + 32768, 1.0, 0.0)[0] == B.ERR_NULL
    torch.cuda.synchronize()


def test_static_entry_point_enqueues_nothing_when_it_refuses_its_arguments():
    """A call that is refused (misaligned or NULL operand) or has nothing to do (M == 0) returns before
    it enqueues anything, also right after a call whose device-side wait ran out; the next good call
    clears the status words on its stream and computes the oracle's result."""
    import torch
    dev = torch.device("cuda:0")
    p = synth.Problem("static_marker", 256, 256, 128, synth.BF16, synth.FP32, 0, 1, 0, 1.0, 0.0, seed=31).generate()
    dA, dB, dC = (harness._to_device(x, dev) for x in (p.A, p.B, p.C))
    desc = harness.desc_of(p)
    # leave a timeout record in the shared status array ...
    assert B.exo_gemm_debug_set(None, 20, 0) == B.OK
    st, detail = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.0, 0, blocking=True)
    assert st == B.ERR_DEVICE_TIMEOUT and detail[0] == 1, (st, detail)
    # ... refused calls do not touch it (they return before anything is enqueued) ...
    assert B.exo_gemm_run_static(desc, dA.data_ptr() + 2, dB.data_ptr(), dC.data_ptr(), 1.0, 0.0)[0] == B.ERR_ALIGNMENT
    assert B.exo_gemm_run_static(desc, 0, dB.data_ptr(), dC.data_ptr(), 1.0, 0.0)[0] == B.ERR_NULL
    empty = B.make_desc(0, 256, 128, synth.BF16, synth.FP32, 0, 1, 0)
    assert B.exo_gemm_run_static(empty, 0, 0, 0, 1.0, 0.0, 0, blocking=True) == (B.OK, [0] * 8)
    torch.cuda.synchronize(dev)
    # ... and the next good call clears it and computes correctly
    dC.copy_(torch.from_numpy(p.C.view(np.uint8)))
    st, detail = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.0, 0, blocking=True)
    assert st == B.OK and detail[0] == 0, (st, detail)
    got = oracle.logical_view(dC.cpu().numpy().view(np.float32), p.M, p.N, 0, p.ldc, synth.FP32)
    assert oracle.max_error(got, *oracle.gemm_problem(p)) <= TOL


def test_static_entry_point_recovers_after_a_timed_out_call():
    """The status array keeps the words of a call whose device-side wait gave up; the next call clears
    them on its stream before its kernel, whose roles read them only after the stream's earlier work is
    complete.  Two good calls after a bad one give the bits of the plan-based entry point."""
    import torch
    dev = torch.device("cuda:0")
    p = synth.Problem("static_after_timeout", 1000, 520, 1032, synth.BF16, synth.FP32, 0, 1, 0, 1.0, 0.0, seed=33).generate()
    want_buf, _ = harness.gemm_host(p, B.flag_split_k(1))
    dA, dB, dC = (harness._to_device(x, dev) for x in (p.A, p.B, p.C))
    desc = harness.desc_of(p)
    stream = torch.cuda.current_stream(dev).cuda_stream
    assert B.exo_gemm_debug_set(None, 20, 3) == B.OK    # CTA 0's producer leaves out its k-block 3: a wait runs out after 20 ms
    st, detail = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.0, stream, blocking=True)
    assert st == B.ERR_DEVICE_TIMEOUT and detail[0] == 1 and detail[5] == 0, (st, detail)
    for blocking in (False, True):                       # back to back, no host sync before the first
        dC.copy_(torch.from_numpy(p.C.view(np.uint8)))
        st, detail = B.exo_gemm_run_static(desc, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.0, stream,
                                           blocking=blocking)
        assert st == B.OK and (detail is None or detail[0] == 0), (st, detail)
        torch.cuda.synchronize(dev)
        assert np.array_equal(dC.cpu().numpy().view(np.float32), want_buf)
