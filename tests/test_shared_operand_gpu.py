"""Parity of the shared-operand cluster variant (two CTA pairs per cluster, the A rows they have in
common fetched half by each and multicast to both; the paper's Section 6 cluster kernels share an
operand the same way) against the CPU oracle, through the C ABI.

Both ways a slot of four CTAs can run are covered: as one 4-CTA cluster (preferred) and as two plain
pairs (what the device substitutes where no four SMs of a GPC are free; forced here for every slot).
With the K split switched off, all of them add the k-blocks of a tile in the same order as the plain
pair kernel, so the three results must also agree bit for bit.

The variant lives in a library of its own; where a deployment leaves it out these tests are skipped.
Tolerance: max |C - Cref| / (sum_k |a b| + |beta c|) <= 1e-3, widened by half an ulp of a 16-bit
output type as in the main parity file.
"""
import numpy as np
import pytest

import oracle
from paper_2609_16389_b200 import binding as B
from paper_2609_16389_b200 import harness, synth
from paper_2609_16389_b200.synth import BF16, FP16, FP32

pytestmark = pytest.mark.gpu
TOL = 1e-3
NO_SPLIT = B.flag_split_k(1)


@pytest.fixture(autouse=True)
def _needs_variant():
    if not B.exo_gemm_has_shared_operand_clusters():
        pytest.skip("this deployment carries the base library only")


def run(p, flags, flags2):
    cbuf, info = harness.gemm_host(p, flags, flags2=flags2)
    return cbuf, oracle.logical_view(cbuf, p.M, p.N, p.c_layout, p.ldc, p.c_dtype), info


def assert_parity(p, got, info):
    cref, den = oracle.gemm_problem(p)
    gate = TOL * den + oracle.output_rounding_slack(cref, p.c_dtype)
    bad = np.abs(got - cref) > gate
    assert not bad.any(), (p.name, int(bad.sum()), np.argwhere(bad)[:5], info)


# M, N, K, ab, cd, la, lb, lc, alpha, beta, extra flags
CASES = [
    (512, 1024, 256, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                       # 2 x 2 slots, nothing ragged
    (300, 700, 200, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                        # ragged M, N and K
    (256, 256, 512, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                        # second tile of the slot entirely outside C
    (260, 8, 72, FP16, FP16, 0, 1, 0, 1.0, 0.0, 0),                           # a sliver
    (512, 1280, 384, BF16, BF16, 0, 1, 0, 1.5, -0.75, 0),                     # 16-bit output, beta
    (520, 1000, 264, BF16, FP32, 1, 0, 0, 1.0, 0.5, 0),                       # A with M contiguous, B with N contiguous
    (640, 900, 320, FP16, FP32, 0, 1, 1, -1.0, 1.0, 0),                       # column-major C (operands swap)
    (768, 1536, 1024, FP16, FP16, 0, 1, 0, 1.0, 0.0, B.flag_k_subblocks(2)),  # two sub-blocks per stage
    (512, 1024, 520, FP32, FP32, 0, 1, 0, 1.0, 0.0, 0),                       # tf32 operands
    (512, 1024, 264, FP32, FP32, 1, 0, 0, 1.0, 0.0, 0),                       # tf32, A with M contiguous: two 32-row boxes each
    (2048, 4096, 512, BF16, FP32, 0, 1, 0, 1.0, 0.0, B.flag_grid_limit(8)),   # persistent: 64 slots' worth of tiles on 2 slots
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c[:3]))
def test_both_slot_forms_match_the_oracle_and_the_pair_kernel(case):
    M, N, K, ab, cd, la, lb, lc, alpha, beta, extra = case
    p = synth.Problem("share", M, N, K, ab, cd, la, lb, lc, alpha, beta, seed=M + 3 * N + K,
                      dist="normal" if ab == FP16 else "uniform").generate()
    flags = NO_SPLIT | extra
    quad_bits, quad, info = run(p, flags, B.FLAG2_SHARE_ALWAYS)
    assert info["cluster_size"] == 4 and info["cta_group"] == 2 and info["tile_n"] == 256 and info["grid"] % 4 == 0
    if not lc:
        assert info["tiles_m"] == -(-M // 256) and info["tiles_n"] == -(-N // 512)   # a slot covers 256 x 512 of C
    assert_parity(p, quad, info)
    sub_bits, _, info_s = run(p, flags, B.FLAG2_SHARE_SUBSTITUTED)
    assert info_s["cluster_size"] == 4
    assert np.array_equal(sub_bits.view(np.uint8), quad_bits.view(np.uint8))
    pair_bits, _, info_p = run(p, flags | B.flag_cta_group(2) | B.flag_tile_n(256), B.FLAG2_SHARE_NEVER)
    assert info_p["cluster_size"] == 2
    assert np.array_equal(pair_bits.view(np.uint8), quad_bits.view(np.uint8))


@pytest.mark.parametrize("flags2", [B.FLAG2_SHARE_ALWAYS, B.FLAG2_SHARE_SUBSTITUTED])
@pytest.mark.parametrize("split", [0, 3])
def test_tail_slots_cut_along_k(flags2, split):
    # 2 x 20 slots of work on 37 slots of CTAs at most: the 3 left over after one wave are cut along K
    import torch
    p = synth.Problem("share_split", 512, 10240, 2048, BF16, FP32, 0, 1, 0, 1.0, 0.25, seed=5).generate()
    flags = B.flag_split_k(split)
    dp = harness.DeviceProblem(p, flags, flags2=flags2)
    try:
        info = dp.plan.info()
        dp.run()
        torch.cuda.synchronize()
        dp.plan.check()
        bits = dp.result_buffer().copy()
        got = oracle.logical_view(bits, p.M, p.N, 0, p.ldc, FP32)
        rng = np.random.default_rng(1)
        rows, cols = rng.integers(0, p.M, 1 << 14), rng.integers(0, p.N, 1 << 14)
        cref, den = oracle.gemm_problem_entries(p, rows, cols)
        assert oracle.max_error(got[rows, cols], cref, den) <= TOL, info
        assert oracle.freivalds(p, got) <= TOL, info
        if info["grid"] == 148:
            assert info["tail_tiles"] == 3 and info["split_k"] == (3 if split else 2) and info["workspace_bytes"] > 0
        for _ in range(2):   # fixed reduction order: repeated runs of the plan agree bit for bit
            dp.reset_c()
            dp.run()
            assert np.array_equal(dp.result_buffer(), bits)
        dp.plan.check()
    finally:
        dp.close()


@pytest.mark.parametrize("flags2", [B.FLAG2_SHARE_ALWAYS, B.FLAG2_SHARE_SUBSTITUTED])
def test_owning_slice_behind_two_whole_waves_starts_from_the_other_slices_sum(flags2):
    # 3 x 5 = 15 slots of work on 7 slots of CTAs: two whole waves, then one tail slot cut in two; its
    # owners find the partial sums written into their accumulators before their slice starts
    p = synth.Problem("share_preload", 768, 2560, 1024, BF16, FP32, 0, 1, 0, 1.0, 0.5, seed=6).generate()
    flags = B.flag_grid_limit(28) | B.flag_split_k(2)
    bits, got, info = run(p, flags, flags2)
    assert (info["grid"], info["tail_tiles"], info["split_k"]) == (28, 1, 2), info
    assert_parity(p, got, info)
    again, _, _ = run(p, flags, flags2)
    assert np.array_equal(again.view(np.uint8), bits.view(np.uint8))


def test_strided_batch_on_shared_operand_clusters():
    import torch
    M, N, K, batch = 384, 640, 320, 5
    bp = synth.BatchedProblem("share_batch", batch, M, N, K, BF16, BF16, 0, 1, 0, 1.0, 0.5, seed=21).generate()
    dev = torch.device("cuda:0")
    dA, dB, dC = (harness._to_device(x, dev) for x in (bp.A, bp.B, bp.C))
    desc = harness.desc_of(bp, NO_SPLIT, 0, B.FLAG2_SHARE_ALWAYS)
    with B.Plan(desc, batch=(batch, bp.stride_a, bp.stride_b, bp.stride_c)) as plan:
        info = plan.info()
        assert info["cluster_size"] == 4 and info["batch_count"] == batch
        plan.run(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.5, torch.cuda.current_stream(dev).cuda_stream)
        torch.cuda.synchronize(dev)
        plan.check()
    out = dC.cpu().numpy().view(np.uint16)
    for i in range(batch):
        q = bp.matrix(i)
        got = oracle.logical_view(out[i * bp.stride_c:(i + 1) * bp.stride_c], M, N, 0, q.ldc, BF16)
        assert_parity(q, got, info)


def test_timeout_in_a_shared_operand_cluster_is_reported_and_the_plan_recovers():
    import torch
    p = synth.Problem("share_tmo", 512, 1024, 1024, BF16, FP32, 0, 1, 0, 1.0, 0.0, seed=10).generate()
    dp = harness.DeviceProblem(p, NO_SPLIT, flags2=B.FLAG2_SHARE_ALWAYS)
    try:
        # CTA 0 leaves out the loads of its k-block 5 (its half of the shared A rows among them): the
        # MMA issuers of both pairs of its cluster run out of time after 20 ms and every role returns
        assert B.exo_gemm_debug_set(dp.plan.handle, 20, 5) == B.OK
        dp.run()
        torch.cuda.synchronize()
        st, detail = B.exo_gemm_check(dp.plan.handle)
        assert st == B.ERR_DEVICE_TIMEOUT and detail[0] == 1, detail
        dp.reset_c()
        dp.run()
        torch.cuda.synchronize()
        dp.plan.check()
        got = oracle.logical_view(dp.result_buffer(), p.M, p.N, 0, p.ldc, FP32)
        cref, den = oracle.gemm_problem(p)
        assert oracle.max_error(got, cref, den) <= TOL
    finally:
        dp.close()


def test_large_square_sampled():
    p = synth.Problem("share_4096", 4096, 4096, 4096, BF16, BF16, 0, 1, 0, 1.0, 0.0, seed=2).generate()
    _, got, info = run(p, 0, B.FLAG2_SHARE_ALWAYS)
    rng = np.random.default_rng(3)
    rows, cols = rng.integers(0, 4096, 1 << 14), rng.integers(0, 4096, 1 << 14)
    cref, den = oracle.gemm_problem_entries(p, rows, cols)
    gate = TOL * den + oracle.output_rounding_slack(cref, BF16)
    assert (np.abs(got[rows, cols] - cref) <= gate).all(), info
    assert oracle.freivalds(p, got) <= TOL + 2.0 ** -8, info
