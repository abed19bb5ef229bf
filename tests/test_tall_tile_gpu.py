"""Parity of the tall 2-CTA tile (256 rows of C per CTA, 512 x 256 per CTA pair: both TMEM accumulators
of a CTA belong to one tile and are multiplied with the same B block) against the CPU oracle, through
the C ABI.  The operation is the same GEMM (the paper's Section 6 kernels differ from one another in
exactly this kind of tile-shape choice), so the same tolerance applies:

    max |C - Cref| / (sum_k |a b| + |beta c|) <= 1e-3,

widened by half an ulp of a 16-bit output type as in the main parity file.  With the K split switched
off the tall tile adds the k-blocks of every output element in the same order as the 128-row kernel, so
the two results must also agree bit for bit.
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
TALL = B.flag2_cta_rows(256)
REGULAR = B.flag2_cta_rows(128) | B.FLAG2_SHARE_NEVER


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
    (512, 256, 256, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                        # exactly one pair tile
    (1024, 512, 512, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                       # 2 x 2 tiles
    (700, 300, 200, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                        # ragged M, N and K
    (130, 256, 512, BF16, FP32, 0, 1, 0, 1.0, 0.0, 0),                        # second accumulator: 2 valid rows; CTA 1 idle
    (257, 40, 72, FP16, FP16, 0, 1, 0, 1.0, 0.0, 0),                          # one row into the second CTA
    (1, 8, 8, BF16, FP32, 0, 1, 0, 2.0, 0.0, 0),
    (1280, 512, 384, BF16, BF16, 0, 1, 0, 1.5, -0.75, 0),                     # 16-bit output, beta
    (1000, 520, 264, BF16, FP32, 1, 0, 0, 1.0, 0.5, 0),                       # A with M contiguous (four 64-row boxes)
    (640, 900, 320, FP16, FP32, 0, 1, 1, -1.0, 1.0, 0),                       # column-major C (operands swap)
    (1024, 512, 520, FP32, FP32, 0, 1, 0, 1.0, 0.0, 0),                       # tf32 operands
    (8192, 2048, 512, BF16, FP32, 0, 1, 0, 1.0, 0.0, B.flag_grid_limit(8)),   # persistent: 128 tiles on 4 pairs
    (1536, 768, 1024, FP16, FP16, 0, 1, 0, 1.0, 1.0, B.flag_max_stages(2) | B.flag_epi_buffers(2)),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c[:3]))
def test_tall_tile_matches_the_oracle_and_the_128_row_kernel(case):
    M, N, K, ab, cd, la, lb, lc, alpha, beta, extra = case
    p = synth.Problem("tall", M, N, K, ab, cd, la, lb, lc, alpha, beta, seed=M + 3 * N + K,
                      dist="normal" if ab == FP16 else "uniform").generate()
    bits, got, info = run(p, NO_SPLIT | extra, TALL)
    assert (info["cta_group"], info["tile_m"], info["tile_n"], info["tile_k"]) == (2, 512, 256, 64 if ab != FP32 else 32)
    assert info["tmem_columns"] == 512 and info["smem_bytes"] <= 232448
    if not lc:
        assert info["tiles_m"] == -(-M // 512) and info["tiles_n"] == -(-N // 256)
    assert_parity(p, got, info)
    ref_bits, _, info_r = run(p, NO_SPLIT | extra | B.flag_cta_group(2) | B.flag_tile_n(256), REGULAR)
    assert info_r["tile_m"] == 256
    assert np.array_equal(ref_bits.view(np.uint8), bits.view(np.uint8))


def test_tall_tile_padding_untouched_and_nan_c_ignored_when_beta_is_zero():
    p = synth.Problem("tall_pad", 600, 500, 136, BF16, FP32, 0, 1, 0, 1.0, 0.0, seed=4, ldc=512).generate()
    p.C[:] = np.nan
    bits, got, info = run(p, NO_SPLIT, TALL)
    assert_parity(p, got, info)
    flat = bits.reshape(-1)
    for i in (0, 1, 127, 128, 255, 256, 511, 512, 598):      # the gap after each row is as it was
        assert np.isnan(flat[i * 512 + 500:(i + 1) * 512]).all(), i


@pytest.mark.parametrize("split", [0, 3, 8])
def test_tall_tail_tiles_cut_along_k(split):
    # 5 x 15 = 75 pair tiles: one more than the 74 pairs of a B200, so one tile is cut along K
    import torch
    p = synth.Problem("tall_split", 2560, 3840, 2048, BF16, FP32, 0, 1, 0, 1.0, 0.25, seed=5).generate()
    dp = harness.DeviceProblem(p, B.flag_split_k(split), flags2=TALL)
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
            assert info["tail_tiles"] == 1 and info["split_k"] == (split if split else 2)   # own choice: slices of 1024 k
            assert info["workspace_bytes"] == (info["split_k"] - 1) * 512 * 256 * 4
        for _ in range(2):   # fixed reduction order: repeated runs of the plan agree bit for bit
            dp.reset_c()
            dp.run()
            assert np.array_equal(dp.result_buffer(), bits)
        dp.plan.check()
    finally:
        dp.close()


def test_tall_tile_strided_batch():
    import torch
    M, N, K, batch = 600, 384, 320, 5
    bp = synth.BatchedProblem("tall_batch", batch, M, N, K, BF16, BF16, 0, 1, 0, 1.0, 0.5, seed=21).generate()
    dev = torch.device("cuda:0")
    dA, dB, dC = (harness._to_device(x, dev) for x in (bp.A, bp.B, bp.C))
    desc = harness.desc_of(bp, NO_SPLIT, 0, TALL)
    with B.Plan(desc, batch=(batch, bp.stride_a, bp.stride_b, bp.stride_c)) as plan:
        info = plan.info()
        assert info["tile_m"] == 512 and info["batch_count"] == batch
        plan.run(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), 1.0, 0.5, torch.cuda.current_stream(dev).cuda_stream)
        torch.cuda.synchronize(dev)
        plan.check()
    out = dC.cpu().numpy().view(np.uint16)
    for i in range(batch):
        q = bp.matrix(i)
        got = oracle.logical_view(out[i * bp.stride_c:(i + 1) * bp.stride_c], M, N, 0, q.ldc, BF16)
        assert_parity(q, got, info)


def test_tall_tile_timeout_is_reported_and_the_plan_recovers():
    import torch
    p = synth.Problem("tall_tmo", 1024, 512, 1024, BF16, FP32, 0, 1, 0, 1.0, 0.0, seed=10).generate()
    dp = harness.DeviceProblem(p, NO_SPLIT, flags2=TALL)
    try:
        assert B.exo_gemm_debug_set(dp.plan.handle, 20, 5) == B.OK   # CTA 0 leaves out the loads of its k-block 5
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


def test_alpha_zero_and_k_zero_on_the_tall_tile():
    p = synth.Problem("tall_a0", 700, 300, 128, BF16, FP32, 0, 1, 0, 0.0, 0.5, seed=8).generate()
    _, got, info = run(p, 0, TALL)
    assert_parity(p, got, info)
    p = synth.Problem("tall_k0", 700, 300, 0, BF16, FP32, 0, 1, 0, 1.0, -2.0, seed=9).generate()
    _, got, info = run(p, 0, TALL)
    assert_parity(p, got, info)


def test_long_k_problem_takes_the_tall_tile_by_default():
    # 4608 x 4096 x 16384: the library's own choice; checked on sampled entries and with the whole-matrix Freivalds test
    p = synth.Problem("tall_auto", 4608, 4096, 16384, BF16, BF16, 0, 1, 0, 1.0, 0.0, seed=2).generate()
    _, got, info = run(p, 0, 0)
    if info["sm_count"] == 148:
        assert info["tile_m"] == 512, info
    rng = np.random.default_rng(3)
    rows, cols = rng.integers(0, 4608, 1 << 14), rng.integers(0, 4096, 1 << 14)
    cref, den = oracle.gemm_problem_entries(p, rows, cols)
    gate = TOL * den + oracle.output_rounding_slack(cref, BF16)
    assert (np.abs(got[rows, cols] - cref) <= gate).all(), info
    assert oracle.freivalds(p, got) <= TOL + 2.0 ** -8, info
