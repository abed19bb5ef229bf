"""Pins for the CPU oracle: what the mathematics fixes, independent of the oracle.

Each test would fail under a plausible oracle mistake: a dropped alpha/beta
term, a transposed operand, a wrong layout index, a wrong 16-bit decode, a
denominator without the beta term, a k loop off by one.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2609_16389_b200 import synth
from paper_2609_16389_b200.synth import BF16, FP16, FP32, ROW_MAJOR, COL_MAJOR

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tiny_gemm_cases.txt")


def run(a, b, c, ab_dtype, c_dtype, alpha, beta, la=ROW_MAJOR, lb=ROW_MAJOR, lc=ROW_MAJOR,
        lda=None, ldb=None, ldc=None, pad=None):
    """a, b, c are logical real arrays; they are rounded to storage, laid out, and run."""
    M, K = a.shape
    N = b.shape[1]
    A = synth.store(synth.round_to_storage(a, ab_dtype), la, lda, pad)
    B = synth.store(synth.round_to_storage(b, ab_dtype), lb, ldb, pad)
    cpad = None if pad is None else (np.float32(np.nan) if c_dtype == FP32 else pad)
    C = synth.store(synth.round_to_storage(c, c_dtype), lc, ldc, cpad)
    lda = lda or synth.min_ld(M, K, la)
    ldb = ldb or synth.min_ld(K, N, lb)
    ldc = ldc or synth.min_ld(M, N, lc)
    return oracle.gemm(M, N, K, A, B, C, ab_dtype, c_dtype, la, lb, lc, lda, ldb, ldc, alpha, beta)


def small_ints(rng, shape, lo=-8, hi=8):
    return rng.integers(lo, hi + 1, size=shape).astype(np.float64)


# ---------------------------------------------------------------- decoders
def test_widen_bf16_and_fp16_known_bit_patterns():
    w = oracle.lib().oracle_widen
    # bf16: sign | 8 exp | 7 frac
    assert w(0x3F80, BF16) == 1.0
    assert w(0xBF80, BF16) == -1.0
    assert w(0x4049, BF16) == 3.140625          # 0x40490000 as fp32
    assert w(0x0000, BF16) == 0.0
    assert w(0x3B80, BF16) == 2.0 ** -8
    # fp16: sign | 5 exp | 10 frac
    assert w(0x3C00, FP16) == 1.0
    assert w(0xC000, FP16) == -2.0
    assert w(0x7BFF, FP16) == 65504.0           # largest finite half
    assert w(0x0001, FP16) == 2.0 ** -24        # smallest subnormal
    assert w(0x03FF, FP16) == 1023 * 2.0 ** -24 # largest subnormal
    assert w(0x0400, FP16) == 2.0 ** -14        # smallest normal
    assert w(0x3555, FP16) == 0.333251953125
    assert w(np.float32(0.1).view(np.uint32).item(), FP32) == float(np.float32(0.1))


def test_widen_fp16_all_finite_patterns_match_numpy():
    bits = np.arange(0, 0x7C00, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    w = oracle.lib().oracle_widen
    step = 7  # every 7th pattern plus the ends: covers all exponents and many fractions
    for b in list(bits[::step]) + [0x7BFF, 0x0400, 0x03FF]:
        assert w(int(b), FP16) == want[int(b)]
        assert w(int(b) | 0x8000, FP16) == -want[int(b)]
    assert np.array_equal(oracle.widen(bits, FP16), want)


def test_numpy_widen_bf16_matches_c_decoder():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 0x7F80, size=2000).astype(np.uint16)
    got = oracle.widen(bits, BF16)
    w = oracle.lib().oracle_widen
    for b, g in zip(bits[:300], got[:300]):
        assert w(int(b), BF16) == g


# ---------------------------------------------------------------- hand-expanded cases
def _golden_cases():
    cases, cur = [], None
    for ln in open(GOLDEN):
        ln = ln.strip()
        if not ln or ln.startswith("#"):
            continue
        t = ln.split()
        if t[0] == "case":
            cur = {"name": t[1]}
            for kv in t[2:]:
                k, v = kv.split("=")
                cur[k] = float(Fraction(v))
            cases.append(cur)
        else:
            cur[t[0]] = np.array([float(Fraction(x)) for x in t[1:]])
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
@pytest.mark.parametrize("ab_dtype", [BF16, FP16])
@pytest.mark.parametrize("layouts", [(0, 0, 0), (1, 1, 1), (0, 1, 0), (1, 0, 1)])
def test_hand_expanded_cases(case, ab_dtype, layouts):
    M, N, K = int(case["M"]), int(case["N"]), int(case["K"])
    a = case["A"].reshape(M, K)
    b = case["B"].reshape(K, N)
    c = case["C"].reshape(M, N)
    la, lb, lc = layouts
    cref, den = run(a, b, c, ab_dtype, FP32, case["alpha"], case["beta"], la, lb, lc)
    assert np.array_equal(cref, case["R"].reshape(M, N))
    assert np.array_equal(den, case["D"].reshape(M, N))


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("ab_dtype", [BF16, FP16])
def test_identity_left_and_right(ab_dtype):
    rng = np.random.default_rng(2)
    n, m = 37, 21
    b = small_ints(rng, (n, m)) / 4.0
    c = small_ints(rng, (n, m)) / 8.0
    cref, den = run(np.eye(n), b, c, ab_dtype, FP32, 2.0, -0.5, lb=COL_MAJOR)
    assert np.array_equal(cref, 2.0 * b - 0.5 * c)
    assert np.array_equal(den, np.abs(b) + np.abs(0.5 * c))
    a = small_ints(rng, (m, n)) / 4.0
    c2 = small_ints(rng, (m, n))
    cref, den = run(a, np.eye(n), c2, ab_dtype, FP32, 1.0, 0.0, la=COL_MAJOR)
    assert np.array_equal(cref, a)
    assert np.array_equal(den, np.abs(a))


def test_permutation_rows_and_columns():
    rng = np.random.default_rng(3)
    n, m = 29, 17
    perm = rng.permutation(n)
    P = np.zeros((n, n))
    P[np.arange(n), perm] = 1.0          # (P B)_i = B_perm[i]
    b = small_ints(rng, (n, m))
    cref, _ = run(P, b, np.zeros((n, m)), BF16, FP32, 1.0, 0.0)
    assert np.array_equal(cref, b[perm])
    a = small_ints(rng, (m, n))
    Q = np.zeros((n, n))
    Q[perm, np.arange(n)] = 1.0          # (A Q)_:,j = A_:,perm[j]
    cref, _ = run(a, Q, np.zeros((m, n)), FP16, FP32, 1.0, 0.0, lb=COL_MAJOR)
    assert np.array_equal(cref, a[:, perm])


def test_rank_one_outer_product():
    rng = np.random.default_rng(4)
    M, N, K, k0 = 19, 23, 11, 7
    u = small_ints(rng, M, -31, 31) / 16.0
    v = small_ints(rng, N, -31, 31) / 32.0
    a = np.zeros((M, K))
    b = np.zeros((K, N))
    a[:, k0] = u
    b[k0, :] = v
    cref, den = run(a, b, np.zeros((M, N)), BF16, FP32, 1.0, 0.0, la=COL_MAJOR, lb=ROW_MAJOR)
    assert np.array_equal(cref, np.outer(u, v))
    assert np.array_equal(den, np.abs(np.outer(u, v)))


@pytest.mark.parametrize("K", [1, 2, 255, 256, 1000, 4099])
def test_all_ones_gives_exactly_K(K):
    M, N = 5, 6
    cref, den = run(np.ones((M, K)), np.ones((K, N)), np.ones((M, N)), BF16, FP32, 1.0, 0.0)
    assert np.all(cref == K) and np.all(den == K)
    cref, den = run(np.ones((M, K)), np.ones((K, N)), np.ones((M, N)), FP16, FP32, 0.5, 1.0)
    assert np.all(cref == K / 2 + 1) and np.all(den == K + 1)


def test_k_zero_and_empty_dims():
    c = np.full((3, 4), 2.0)
    cref, den = run(np.zeros((3, 0)), np.zeros((0, 4)), c, BF16, FP32, 3.0, 0.5)
    assert np.all(cref == 1.0) and np.all(den == 1.0)
    cref, den = run(np.zeros((0, 5)), np.zeros((5, 4)), np.zeros((0, 4)), BF16, FP32, 1.0, 0.0)
    assert cref.shape == (0, 4)


def test_alternating_signs_cancel_but_denominator_does_not():
    K = 64
    a = np.ones((2, K))
    b = np.tile(np.array([[1.0], [-1.0]]), (K // 2, 3))
    cref, den = run(a, b, np.zeros((2, 3)), BF16, FP32, 1.0, 0.0)
    assert np.all(cref == 0.0) and np.all(den == K)


# ---------------------------------------------------------------- invariants
def _random_problem(rng, M, N, K, dtype):
    scale = 64.0
    return (small_ints(rng, (M, K), -64, 64) / scale, small_ints(rng, (K, N), -64, 64) / scale,
            small_ints(rng, (M, N), -64, 64) / scale)


@pytest.mark.parametrize("ab_dtype,c_dtype", [(BF16, FP32), (FP16, FP16), (BF16, BF16)])
def test_layout_and_leading_dimension_invariance_bitwise(ab_dtype, c_dtype):
    rng = np.random.default_rng(5)
    M, N, K = 13, 9, 21
    a, b, c = _random_problem(rng, M, N, K, ab_dtype)
    base = run(a, b, c, ab_dtype, c_dtype, 1.5, -2.0)
    nan16 = np.uint16(0x7FC1 if ab_dtype == BF16 else 0x7E01)
    for la in (0, 1):
        for lb in (0, 1):
            for lc in (0, 1):
                got = run(a, b, c, ab_dtype, c_dtype, 1.5, -2.0, la, lb, lc)
                assert np.array_equal(got[0], base[0]) and np.array_equal(got[1], base[1])
                padded = run(a, b, c, ab_dtype, c_dtype, 1.5, -2.0, la, lb, lc,
                             lda=32, ldb=40, ldc=24, pad=nan16)
                assert np.array_equal(padded[0], base[0]) and np.array_equal(padded[1], base[1])


def test_transpose_invariant_bitwise():
    rng = np.random.default_rng(6)
    M, N, K = 14, 10, 33
    a, b, c = _random_problem(rng, M, N, K, BF16)
    cref, den = run(a, b, c, BF16, FP32, 0.75, 1.25)
    cref_t, den_t = run(b.T.copy(), a.T.copy(), c.T.copy(), BF16, FP32, 0.75, 1.25)
    assert np.array_equal(cref_t, cref.T) and np.array_equal(den_t, den.T)


def test_linearity_in_alpha_beta_and_beta_zero_ignores_nan():
    rng = np.random.default_rng(7)
    M, N, K = 11, 12, 50
    a, b, c = _random_problem(rng, M, N, K, FP16)
    s, d = run(a, b, c, FP16, FP32, 1.0, 0.0)
    got, den = run(a, b, c, FP16, FP32, -3.0, 0.25)
    assert np.allclose(got, -3.0 * s + 0.25 * c, rtol=0, atol=1e-12)
    assert np.allclose(den, d + np.abs(0.25 * c), rtol=0, atol=1e-12)
    # beta == 0: C_in must not be read at all
    A = synth.store(synth.round_to_storage(a, FP16), ROW_MAJOR)
    B = synth.store(synth.round_to_storage(b, FP16), ROW_MAJOR)
    Cnan = np.full(M * N, np.nan, dtype=np.float32)
    got0, _ = oracle.gemm(M, N, K, A, B, Cnan, FP16, FP32, 0, 0, 0, K, N, N, 1.0, 0.0)
    assert np.array_equal(got0, s)


@pytest.mark.parametrize("shape", [(64, 48, 80), (130, 70, 257), (33, 512, 100)])
@pytest.mark.parametrize("ab_dtype,dist", [(BF16, "uniform"), (FP16, "normal")])
def test_against_float64_library_matmul(shape, ab_dtype, dist):
    M, N, K = shape
    p = synth.Problem("t", M, N, K, ab_dtype, FP32, ROW_MAJOR, COL_MAJOR, ROW_MAJOR, 0.5, 1.0,
                      seed=99, dist=dist).generate()
    cref, den = oracle.gemm_problem(p)
    A = oracle.logical_view(p.A, M, K, p.a_layout, p.lda, ab_dtype)
    B = oracle.logical_view(p.B, K, N, p.b_layout, p.ldb, ab_dtype)
    C = oracle.logical_view(p.C, M, N, p.c_layout, p.ldc, FP32)
    want = 0.5 * (A @ B) + C
    wden = np.abs(A) @ np.abs(B) + np.abs(C)
    assert np.max(np.abs(cref - want) / wden) < 1e-13
    assert np.max(np.abs(den - wden) / wden) < 1e-13


def test_rows_and_entries_agree_with_full_bitwise():
    p = synth.Problem("t", 70, 45, 130, BF16, BF16, COL_MAJOR, ROW_MAJOR, COL_MAJOR, 1.0, 0.5,
                      seed=5).generate()
    cref, den = oracle.gemm_problem(p)
    band, bden = oracle.gemm_problem(p, rows=(17, 40))
    assert np.array_equal(band, cref[17:40]) and np.array_equal(bden, den[17:40])
    rng = np.random.default_rng(8)
    r = rng.integers(0, 70, 200)
    c = rng.integers(0, 45, 200)
    e, ed = oracle.gemm_problem_entries(p, r, c)
    assert np.array_equal(e, cref[r, c]) and np.array_equal(ed, den[r, c])


# ---------------------------------------------------------------- the metric itself
def test_metric_flags_a_single_bad_entry_and_passes_a_small_one():
    p = synth.Problem("t", 40, 30, 64, BF16, FP32, 0, 1, 0, 1.0, 0.0, seed=3).generate()
    cref, den = oracle.gemm_problem(p)
    bad = cref.copy()
    bad[7, 9] += 2e-3 * den[7, 9]
    r = oracle.error_ratio(bad, cref, den)
    assert np.argmax(r) == 7 * 30 + 9 and abs(r[7, 9] - 2e-3) < 1e-9
    assert oracle.max_error(bad, cref, den) > oracle.TOLERANCE
    ok = cref.copy()
    ok[7, 9] += 0.5e-3 * den[7, 9]
    assert oracle.max_error(ok, cref, den) < oracle.TOLERANCE
    z = np.zeros((2, 2))
    assert oracle.max_error(z, z, z) == 0.0
    assert oracle.max_error(z + 1e-30, z, z) == np.inf
    nanc = cref.copy()
    nanc[0, 0] = np.nan
    assert oracle.max_error(nanc, cref, den) == np.inf


def test_output_rounding_slack_is_half_an_ulp_of_the_output_type():
    """The widened gate of the 16-bit-output tests: slack = u_out * |Cref| with u_out = 2^-8 (bf16),
    2^-11 (fp16), 0 (fp32).  Pinned against the spacing of the output type itself: at a point halfway
    between two neighbouring representable values the slack covers the half ulp a correctly rounded
    result is off by, and stays below a whole ulp -- twice or half the constant fails one of the two."""
    def bf16_value(bits):
        return float((np.array([bits], np.uint32) << np.uint32(16)).view(np.float32)[0])
    for e in (-3, 0, 1, 8, 11):                      # binades [2^e, 2^(e+1))
        for frac in (0, 1, 37, 127):                 # of the 7 stored fraction bits
            bits = ((127 + e) << 7) | frac
            lo, hi = bf16_value(bits), bf16_value(bits + 1)
            ulp, mid = hi - lo, 0.5 * (lo + hi)
            for sign in (1.0, -1.0):
                slack = float(oracle.output_rounding_slack(np.array([sign * mid]), BF16)[0])
                assert 0.5 * ulp <= slack < ulp, (e, frac, slack, ulp)
    for x16 in (np.float16(1.0), np.float16(0.3333), np.float16(2048.0), np.float16(3.0e-3), np.float16(60000.0)):
        lo, ulp = float(x16), float(np.spacing(x16))
        mid = lo + 0.5 * ulp
        slack = float(oracle.output_rounding_slack(np.array([-mid]), FP16)[0])
        assert 0.5 * ulp <= slack < ulp, (x16, slack, ulp)
    # fp16 results below the smallest normal number (2^-14): the spacing is 2^-24 whatever the value
    for x16 in (np.float16(9.0e-6), np.float16(6.0e-5), np.float16(6.0e-8), np.float16(3.0e-7)):
        lo, ulp = float(x16), float(np.spacing(x16))
        assert ulp == 2.0 ** -24 and lo < 2.0 ** -14
        slack = float(oracle.output_rounding_slack(np.array([-(lo + 0.5 * ulp)]), FP16)[0])
        assert 0.5 * ulp <= slack < ulp, (x16, slack, ulp)
    assert float(oracle.output_rounding_slack(np.array([0.0]), FP16)[0]) == 0.0
    assert np.all(oracle.output_rounding_slack(np.array([1.0, -257.0, 1e30]), FP32) == 0.0)
    # the gate as the GPU tests apply it, on an all-positive sum that is a bf16 tie: K = 257 ones.
    # Cref = Den = 257 lies halfway between 256 and 258; the correctly rounded result (either
    # neighbour) is off by 1 = half an ulp, which the literal 1e-3 * Den = 0.257 rejects and the
    # widened gate accepts; a result one whole ulp further away is rejected.
    K = 257
    cref, den = run(np.ones((3, K)), np.ones((K, 2)), np.zeros((3, 2)), BF16, BF16, 1.0, 0.0)
    assert np.all(cref == K) and np.all(den == K)
    rounded = oracle.widen(synth.round_to_storage(cref.astype(np.float32), BF16), BF16)   # storage rounding, not the oracle's
    assert set(np.unique(rounded)) <= {256.0, 258.0}
    gate = oracle.TOLERANCE * den + oracle.output_rounding_slack(cref, BF16)
    assert np.all(np.abs(rounded - cref) > oracle.TOLERANCE * den)
    assert np.all(np.abs(rounded - cref) <= gate)
    for wrong in (254.0, 260.0):
        assert np.all(np.abs(wrong - cref) > gate)


def test_freivalds_accepts_truth_and_catches_a_corrupted_tile():
    p = synth.Problem("t", 96, 80, 128, FP16, FP32, 0, 0, 0, 0.5, 1.0, seed=4, dist="normal").generate()
    cref, den = oracle.gemm_problem(p)
    assert oracle.freivalds(p, cref) < 1e-12
    bad = cref.copy()
    bad[32:64, 16:48] = 0.0
    assert oracle.freivalds(p, bad) > oracle.TOLERANCE


# ---------------------------------------------------------------- the generator
def test_generator_is_layout_independent_and_seeded():
    a = synth.matrix(11, synth.TAG_A, 50, 70, BF16)
    b = synth.matrix(11, synth.TAG_A, 50, 70, BF16, chunk_rows=7)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, synth.matrix(12, synth.TAG_A, 50, 70, BF16))
    assert not np.array_equal(a, synth.matrix(11, synth.TAG_B, 50, 70, BF16))
    for layout in (0, 1):
        for ld in (None, 96):
            buf = synth.store(a, layout, ld)
            ld_eff = ld or synth.min_ld(50, 70, layout)
            assert np.array_equal(synth.load(buf, 50, 70, layout, ld_eff), a)


def test_generator_statistics():
    rows, cols = np.arange(400), np.arange(500)
    u = synth.uniform_pm1(7, 1, rows, cols).astype(np.float64)
    assert u.min() >= -1.0 and u.max() < 1.0
    assert abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.01
    hist, _ = np.histogram(u, bins=16, range=(-1, 1))
    assert hist.min() > 0.9 * u.size / 16 and hist.max() < 1.1 * u.size / 16
    # neighbouring entries are uncorrelated
    assert abs(np.corrcoef(u[:, :-1].ravel(), u[:, 1:].ravel())[0, 1]) < 0.01
    assert abs(np.corrcoef(u[:-1].ravel(), u[1:].ravel())[0, 1]) < 0.01
    z = synth.normal_01(7, 1, rows, cols)
    assert abs(z.mean()) < 0.01 and abs(z.var() - 1.0) < 0.02
    assert abs((np.abs(z) < 1.0).mean() - 0.6827) < 0.01


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, 1.0 + 2 ** -8 + 2 ** -20,
                  -1.0 - 2 ** -8, 0.0, 2.0 ** -20], dtype=np.float32)
    got = oracle.widen(synth.f32_to_bf16_bits(x), BF16)
    want = np.array([1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, 1.0 + 2 ** -7, -1.0, 0.0, 2.0 ** -20])
    assert np.array_equal(got, want)


def test_tf32_grid_rounding_and_fp32_operands_in_the_oracle():
    x = np.array([1.0, 1.0 + 2 ** -11, 1.0 + 3 * 2 ** -11, 1.0 + 2 ** -10, -1.0 - 2 ** -11 - 2 ** -20, 3.14159265, 0.0],
                 dtype=np.float32)
    got = synth.f32_round_to_tf32(x)
    want = np.array([1.0, 1.0, 1.0 + 2 ** -9, 1.0 + 2 ** -10, -1.0 - 2 ** -10, 3.140625, 0.0], dtype=np.float32)
    assert np.array_equal(got, want)                       # ties to even, 10 fraction bits kept
    assert np.all(got.view(np.uint32) & 0x1FFF == 0)
    # fp32 operands go through the same definition: an all-ones product gives exactly K
    M, N, K = 5, 4, 300
    A = np.ones(M * K, np.float32)
    Bm = np.ones(K * N, np.float32)
    C = np.zeros(M * N, np.float32)
    cref, den = oracle.gemm(M, N, K, A, Bm, C, FP32, FP32, 0, 0, 0, K, N, N, 1.0, 0.0)
    assert np.all(cref == K) and np.all(den == K)
    p = synth.Problem("t32", 40, 24, 64, FP32, FP32, 0, 1, 0, 0.5, 1.0, seed=9).generate()
    assert np.all(p.A.view(np.uint32) & 0x1FFF == 0) and np.any(p.C.view(np.uint32) & 0x1FFF != 0)
    cref, den = oracle.gemm_problem(p)
    A64 = oracle.logical_view(p.A, 40, 64, 0, p.lda, FP32)
    B64 = oracle.logical_view(p.B, 64, 24, 1, p.ldb, FP32)
    C64 = oracle.logical_view(p.C, 40, 24, 0, p.ldc, FP32)
    assert np.max(np.abs(cref - (0.5 * (A64 @ B64) + C64))) < 1e-12


def test_gemv_oracle_against_closed_forms_and_a_library_product():
    rng = np.random.default_rng(12)
    M, N, lda = 37, 53, 60
    A = np.full(M * lda, np.nan, dtype=np.float32)                # padding must never be read
    Al = rng.integers(-8, 9, size=(M, N)).astype(np.float32) / 4
    A.reshape(M, lda)[:, :N] = Al
    x = (rng.integers(-8, 9, size=N) / 8).astype(np.float32)
    y = rng.integers(-8, 9, size=M).astype(np.float32)
    yref, den = oracle.gemv(M, N, A, lda, x, y, 2.0, -0.5)
    want = 2.0 * (Al.astype(np.float64) @ x.astype(np.float64)) - 0.5 * y
    assert np.array_equal(yref, want)                              # small dyadic values: exact either way
    assert np.array_equal(den, np.abs(Al.astype(np.float64)) @ np.abs(x.astype(np.float64)) + np.abs(0.5 * y))
    ones = np.ones(M * lda, np.float32)
    yref, den = oracle.gemv(M, N, ones, lda, np.ones(N, np.float32), np.full(M, np.nan, np.float32), 1.0, 0.0)
    assert np.all(yref == N) and np.all(den == N)                  # beta == 0 ignores y
    e = np.zeros(N, np.float32); e[7] = 1.0                        # unit vector picks a column
    yref, _ = oracle.gemv(M, N, A, lda, e, y, 1.0, 0.0)
    assert np.array_equal(yref, Al[:, 7].astype(np.float64))
    # as a one-column GEMM the fp16 oracle gives the same numbers on fp16-exact data
    A16 = synth.round_to_storage(Al, FP16); x16 = synth.round_to_storage(x.reshape(N, 1), FP16)
    cref, cden = oracle.gemm(M, 1, N, synth.store(A16, 0), synth.store(x16, 0), np.zeros(M, np.float32),
                             FP16, FP32, 0, 0, 0, N, 1, 1, 1.0, 0.0)
    g, gd = oracle.gemv(M, N, A, lda, x, y, 1.0, 0.0)
    assert np.array_equal(cref[:, 0], g) and np.array_equal(cden[:, 0], gd)


def test_gemv_oracle_column_major_against_closed_forms_and_the_gemm_oracle():
    # hand-checked: a_ij = i + 5j (M = 5, N = 3, stored column by column with lda = 7), x = (1, 2, 3), y = 1:
    # row i gives i + 2(i + 5) + 3(i + 10) = 6i + 40; with alpha = 1, beta = 1/2: 6i + 40.5
    M, N, lda = 5, 3, 7
    A = np.full(N * lda, np.nan, dtype=np.float32)                 # padding must never be read
    for j in range(N):
        A[j * lda:j * lda + M] = np.arange(M) + 5 * j
    x = np.array([1, 2, 3], np.float32)
    yref, den = oracle.gemv(M, N, A, lda, x, np.ones(M, np.float32), 1.0, 0.5, layout=1)
    assert np.array_equal(yref, 6.0 * np.arange(M) + 40.5) and np.array_equal(den, 6.0 * np.arange(M) + 40.5)
    # a transposed operand must change the answer (a_ij read as a_ji would give other numbers)
    sq = np.arange(9, dtype=np.float32)                            # 3 x 3: row-major reading vs column-major reading
    r, _ = oracle.gemv(3, 3, sq, 3, x, np.zeros(3, np.float32), 1.0, 0.0, layout=0)
    c, _ = oracle.gemv(3, 3, sq, 3, x, np.zeros(3, np.float32), 1.0, 0.0, layout=1)
    assert np.array_equal(r, [8, 26, 44]) and np.array_equal(c, [24, 30, 36])
    # random dyadic data: equals the row-major oracle on the transposed buffer, numpy in fp64, and the
    # one-column GEMM oracle with a column-major A
    rng = np.random.default_rng(13)
    M, N, lda = 41, 29, 48
    Al = rng.integers(-8, 9, size=(M, N)).astype(np.float32) / 4
    A = np.full(N * lda, np.nan, dtype=np.float32)
    A.reshape(N, lda)[:, :M] = Al.T
    x = (rng.integers(-8, 9, size=N) / 8).astype(np.float32)
    y = rng.integers(-8, 9, size=M).astype(np.float32)
    yref, den = oracle.gemv(M, N, A, lda, x, y, -1.5, 0.25, layout=1)
    assert np.array_equal(yref, -1.5 * (Al.astype(np.float64) @ x.astype(np.float64)) + 0.25 * y)
    assert np.array_equal(den, np.abs(Al.astype(np.float64)) @ np.abs(x.astype(np.float64)) + np.abs(0.25 * y))
    rowbuf = np.ascontiguousarray(Al).reshape(-1)
    yrow, drow = oracle.gemv(M, N, rowbuf, N, x, y, -1.5, 0.25, layout=0)
    assert np.array_equal(yref, yrow) and np.array_equal(den, drow)
    A16 = synth.round_to_storage(Al, FP16); x16 = synth.round_to_storage(x.reshape(N, 1), FP16)
    cref, cden = oracle.gemm(M, 1, N, synth.store(A16, 1), synth.store(x16, 0), np.zeros(M, np.float32),
                             FP16, FP32, 1, 0, 0, M, 1, 1, 1.0, 0.0)
    g, gd = oracle.gemv(M, N, A, lda, x, y, 1.0, 0.0, layout=1)
    assert np.array_equal(cref[:, 0], g) and np.array_equal(cden[:, 0], gd)
