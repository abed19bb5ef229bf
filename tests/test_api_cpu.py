"""Host-side tests of the C-ABI library that need no GPU: the library loads and
exports what the header declares, argument validation, plan preview, and the
persistent tile schedule."""
import ctypes
import os
import re

import pytest

from paper_2609_16389_b200 import binding as B
from paper_2609_16389_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "exo_gemm.h")


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(exo_gem[mv]_[a-z_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    lib = B.lib()
    declared = _declared_functions()
    assert "exo_gemm_create" in declared and "exo_gemm_run" in declared and "exo_gemm_destroy" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in exo_gemm.h but not exported"
    assert set(declared) == set(B.EXPORTED_SYMBOLS)


def test_status_strings():
    for code in range(8):
        assert B.exo_gemm_status_string(code)
    assert B.exo_gemm_status_string(B.OK) == "ok"
    assert "unknown" in B.exo_gemm_status_string(99)


def good(**kw):
    d = dict(M=256, N=192, K=128, ab_dtype=B.BF16, c_dtype=B.FP32, a_layout=0, b_layout=1, c_layout=0)
    d.update(kw)
    return B.make_desc(**d)


def test_validate_accepts_the_supported_set():
    assert B.exo_gemm_validate(good()) == B.OK
    for ab in (B.BF16, B.FP16):
        for cd in (B.FP32, ab):
            for la in (0, 1):
                for lb in (0, 1):
                    for lc in (0, 1):
                        assert B.exo_gemm_validate(good(ab_dtype=ab, c_dtype=cd, a_layout=la, b_layout=lb,
                                                        c_layout=lc)) == B.OK
    assert B.exo_gemm_validate(good(M=0)) == B.OK
    assert B.exo_gemm_validate(good(K=0)) == B.OK
    assert B.exo_gemm_validate(good(M=1000, N=1000, K=1000)) == B.OK
    assert B.exo_gemm_validate(good(lda=136, ldb=160, ldc=200)) == B.OK


def test_validate_rejects_bad_arguments():
    assert B.lib().exo_gemm_validate(None) == B.ERR_NULL
    assert B.exo_gemm_validate(good(M=-1)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(N=2 ** 31)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(ab_dtype=7)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(c_layout=2)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(lda=64)) == B.ERR_INVALID_ARG          # row-major A needs lda >= K
    assert B.exo_gemm_validate(good(ldb=120)) == B.ERR_INVALID_ARG         # col-major B needs ldb >= K
    assert B.exo_gemm_validate(good(ldc=100)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(device=-2)) == B.ERR_INVALID_ARG
    d = good()
    d.flags2 = 12
    assert B.exo_gemm_validate(d) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=3)) == B.ERR_INVALID_ARG                       # cta_group 3
    assert B.exo_gemm_validate(good(flags=B.flag_tile_n(192))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=B.flag_cta_group(2) | B.flag_tile_n(64))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=15 << 28)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=B.flag_max_stages(1))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=B.flag_max_stages(9))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags=B.flag_epi_buffers(3))) == B.ERR_INVALID_ARG


def test_validate_unsupported_but_legal_blas_calls():
    assert B.exo_gemm_validate(good(ab_dtype=B.FP32, c_dtype=B.FP32)) == B.OK        # tf32 mode
    for la, lb in ((1, 1), (0, 0), (1, 0)):                                          # ... in every operand layout
        assert B.exo_gemm_validate(good(ab_dtype=B.FP32, c_dtype=B.FP32, a_layout=la, b_layout=lb)) == B.OK
    assert B.exo_gemm_validate(good(ab_dtype=B.FP32, c_dtype=B.BF16)) == B.ERR_UNSUPPORTED
    assert B.exo_gemm_validate(good(ab_dtype=B.BF16, c_dtype=B.FP16)) == B.ERR_UNSUPPORTED


def test_leading_dimensions_tma_cannot_address_are_repacked():
    """Rows that do not start on 16-byte boundaries are legal: the plan owns an aligned copy of such a matrix
    (its contiguous extent rounded up to 64 elements) and says so; plans without scratch of their own refuse."""
    for kw, want in ((dict(ab_dtype=B.FP32, K=130), 3),          # 520 bytes per row of A and of B
                     (dict(ab_dtype=B.FP32, K=132), 0),
                     (dict(K=100), 3),                           # 200 bytes
                     (dict(K=100, lda=104), 2), (dict(K=100, ldb=104), 1), (dict(K=100, lda=104, ldb=104), 0),
                     (dict(N=190), 4), (dict(N=190, ldc=192), 0),             # fp32 C, ldc = 190
                     (dict(M=250, N=190, K=100, a_layout=1, c_layout=1), 7),   # col-major A (lda = 250), B (100), col-major C (250)
                     (dict(M=0, N=190, K=100), 0), (dict(K=0, lda=3, ldb=5), 0)):    # matrices that are never touched
        d = good(**kw)
        assert B.exo_gemm_validate(d) == B.OK, kw
        st, info = B.exo_gemm_plan_preview(d, 148)
        assert st == B.OK and info.repacked == want, (kw, info.repacked)
    st, info = B.exo_gemm_plan_preview(good(M=256, N=190, K=100), 148)
    # A: 256 rows x 128 bf16, B (K x N col-major): 190 rows x 128 bf16, C: 256 rows x 192 fp32
    assert info.repacked == 7 and info.workspace_bytes == 256 * 128 * 2 + 190 * 128 * 2 + 256 * 192 * 4
    h = ctypes.c_void_p()
    assert B.lib().exo_gemm_create_batched(ctypes.byref(h), ctypes.byref(good(K=100)), 4, 1 << 16, 1 << 16, 1 << 16) == B.ERR_UNSUPPORTED


def test_benchmark_configs_are_in_the_supported_set():
    for idx, var in ((0, None), (1, None), (2, None), (3, "a"), (3, "b")):
        p = synth.config(idx, var)
        d = B.make_desc(p.M, p.N, p.K, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout, p.c_layout,
                        p.lda, p.ldb, p.ldc)
        assert B.exo_gemm_validate(d) == B.OK
    for M in synth.SWEEP_DIMS:
        for N in synth.SWEEP_DIMS:
            for K in synth.SWEEP_DIMS:
                p = synth.sweep_problem(M, N, K)
                d = B.make_desc(p.M, p.N, p.K, p.ab_dtype, p.c_dtype, p.a_layout, p.b_layout, p.c_layout)
                assert B.exo_gemm_validate(d) == B.OK, (M, N, K)


def test_plan_preview_geometry_and_overrides():
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, c_dtype=B.BF16), 148)
    assert st == B.OK
    i = info.as_dict()
    assert i["tile_m"] == 128 * i["cta_group"] and i["tile_k"] in (64, 128)
    st, t32 = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, ab_dtype=B.FP32), 148)
    assert st == B.OK and t32.tile_k in (32, 64)
    assert i["tiles_m"] * i["tile_m"] >= 4096 and i["tiles_n"] * i["tile_n"] >= 4096
    assert i["grid"] <= 148 and i["grid"] % i["cta_group"] == 0
    assert i["smem_bytes"] <= 232448 and i["tmem_columns"] == 2 * i["tile_n"] <= 512
    assert i["kernel_launches_per_run"] == 1 and i["swapped"] == 0
    for g, bn in ((1, 64), (1, 128), (1, 256), (2, 128), (2, 256)):
        st, info = B.exo_gemm_plan_preview(good(M=1000, N=520, K=264,
                                                flags=B.flag_cta_group(g) | B.flag_tile_n(bn)), 148)
        i = info.as_dict()
        assert (i["cta_group"], i["tile_n"]) == (g, bn)
        assert i["tiles_m"] == -(-1000 // (128 * g)) and i["tiles_n"] == -(-520 // bn)
        assert i["grid"] == min(148 // g, i["tiles_m"] * i["tiles_n"]) * g
        assert i["tile_k"] in (64, 128) and i["stages"] >= 2 and i["epilogue_buffers"] in (1, 2)
        assert (i["stages"] * (i["tile_k"] // 64) * (16384 + bn // g * 128) + 32768 * i["epilogue_buffers"] + 1536
                == i["smem_bytes"] <= 232448)
    # column-major C is computed as the transposed product
    st, info = B.exo_gemm_plan_preview(good(M=512, N=2048, K=64, c_layout=1, ldc=512), 148)
    i = info.as_dict()
    assert i["swapped"] == 1 and i["tiles_m"] * i["tile_m"] >= 2048 and i["tiles_n"] * i["tile_n"] >= 512
    # grid limit and band override
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=512, flags=B.flag_grid_limit(8) | B.flag_band(3)
                                            | B.flag_cta_group(2) | B.flag_tile_n(256)), 148)
    assert info.grid == 8 and info.raster_band == 3
    st, info = B.exo_gemm_plan_preview(good(flags=B.flag_max_stages(2) | B.flag_epi_buffers(1)), 148)
    assert info.stages == 2 and info.epilogue_buffers == 1
    st, info = B.exo_gemm_plan_preview(good(M=0), 148)
    assert st == B.OK and info.kernel_launches_per_run == 0
    assert B.exo_gemm_plan_preview(good(), 0)[0] == B.ERR_INVALID_ARG


@pytest.mark.parametrize("tiles_m,tiles_n", [(1, 1), (4, 4), (16, 16), (3, 5), (4, 64), (64, 4), (48, 47), (7, 1)])
@pytest.mark.parametrize("band", [1, 2, 3, 8, 15])
@pytest.mark.parametrize("along_m", [0, 1])
def test_schedule_visits_every_tile_exactly_once(tiles_m, tiles_n, band, along_m):
    for workers in (1, 2, 7, 74, 148):
        seen = {}
        longest, shortest = 0, 10 ** 9
        for w in range(workers):
            seq = B.exo_gemm_schedule_enumerate(tiles_m, tiles_n, band, along_m, workers, w)
            longest, shortest = max(longest, len(seq)), min(shortest, len(seq))
            for t in seq:
                assert 0 <= t[0] < tiles_m and 0 <= t[1] < tiles_n
                assert t not in seen, f"tile {t} visited twice"
                seen[t] = w
        assert len(seen) == tiles_m * tiles_n
        assert longest - shortest <= 1                     # round-robin: balanced to within one tile


def test_schedule_order_is_band_swizzled():
    # 3 x 5 tiles, bands of 2 tile columns: walk a band's columns first, then the next tile row
    seq = B.exo_gemm_schedule_enumerate(3, 5, 2, 0, 1, 0)
    assert seq[:6] == [(0, 0), (0, 1), (1, 0), (1, 1), (2, 0), (2, 1)]
    assert seq[6:12] == [(0, 2), (0, 3), (1, 2), (1, 3), (2, 2), (2, 3)]
    assert seq[12:] == [(0, 4), (1, 4), (2, 4)]                       # narrower last band
    seq = B.exo_gemm_schedule_enumerate(3, 5, 2, 1, 1, 0)              # transposed raster
    assert seq[:4] == [(0, 0), (1, 0), (0, 1), (1, 1)]
    assert seq[-5:] == [(2, 0), (2, 1), (2, 2), (2, 3), (2, 4)]
    # a wave of consecutive indices covers a compact patch: 8 workers on 16x16 tiles, band 4
    first_wave = [B.exo_gemm_schedule_enumerate(16, 16, 4, 0, 8, w)[0] for w in range(8)]
    assert {t[0] for t in first_wave} == {0, 1} and {t[1] for t in first_wave} == {0, 1, 2, 3}
    with pytest.raises(ValueError):
        B.exo_gemm_schedule_enumerate(3, 5, 0, 0, 1, 0)


def test_create_fails_cleanly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st, h = B.exo_gemm_create(good())
    assert st in (B.ERR_CUDA, B.ERR_ARCH) and h is None      # no CPU fallback: an error, not a result
    with pytest.raises(B.ExoGemmError):
        B.Plan(good())
    assert B.exo_gemm_destroy(None) == B.OK
    assert B.exo_gemm_run(None, 0, 0, 0, 1.0, 0.0, 0) == B.ERR_NULL


@pytest.mark.parametrize("tiles,workers,tail_workers", [(256, 74, 68), (256, 74, 74), (256, 74, 0), (32, 148, 128), (5, 148, 40),
                                                        (300, 148, 7), (300, 148, 148), (148, 148, 0), (149, 148, 8),
                                                        (48, 74, 74), (96, 74, 74), (1, 1, 0), (0, 4, 0), (75, 74, 3)])
@pytest.mark.parametrize("nkb", [64, 7, 1000, 192])
@pytest.mark.parametrize("snap", [0, 4, 8])
def test_work_schedule_covers_every_tile_and_k_block_exactly_once(tiles, workers, tail_workers, nkb, snap):
    tail = tiles % workers
    if tail_workers and (tail_workers < tail or tail_workers > tail * nkb or tail == 0):
        pytest.skip("not a plan the library would make")
    cover = {}
    longest = 0
    loads = []
    for w in range(workers):
        items = B.exo_gemm_schedule_work(tiles, workers, tail_workers, nkb, w, snap)
        longest = max(longest, len(items))
        loads.append(sum(e - b for _, _, _, b, e in items))
        for tile, sl, n_sl, b, e in items:
            assert 0 <= tile < tiles and 0 <= b < e <= nkb and 0 <= sl < n_sl
            cover.setdefault(tile, []).append((b, e, sl, n_sl))
        # the order of execution: contributing parts first, whole tiles, owning parts last
        kinds = ["c" if sl > 0 else ("o" if n_sl > 1 else "w") for _, sl, n_sl, _, _ in items]
        assert "".join(kinds).lstrip("c").rstrip("o").strip("w") == "", kinds
    assert sorted(cover) == list(range(tiles))
    for tile, parts in cover.items():
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == nkb
        assert all(parts[i][1] == parts[i + 1][0] for i in range(len(parts) - 1))      # a partition of K
        assert [p[2] for p in parts] == list(range(len(parts)))                         # slice order = K order
        assert all(p[3] == len(parts) for p in parts)                                   # every part knows how many there are
        if tile < tiles - tail or not tail_workers:
            assert len(parts) == 1
    if tail_workers:
        # the tail's k-blocks are shared evenly: nobody holds more than a k-block beyond an even share
        tail_loads = [l - (tiles // workers) * nkb for l in loads]
        share = [l for l in tail_loads[:tail_workers]]
        eff_snap = min(snap, nkb // 8, tail * nkb // tail_workers // 4)
        assert max(share) - min(share) <= 1 + 2 * eff_snap and sum(share) == tail * nkb
        for tile, parts in cover.items():                       # no part shorter than the snap distance
            if len(parts) > 1 and nkb * tail >= tail_workers * (2 * eff_snap + 1):
                assert min(e - b for b, e, _, _ in parts) > eff_snap, (tile, parts)
        assert all(l == 0 for l in tail_loads[tail_workers:])
    assert longest <= tiles // workers + 2


def test_contributing_parts_come_first_and_owning_parts_last():
    # 96 tiles on 74 workers with 192 k-blocks each: one whole wave, then 22 tiles whose 4224 k-blocks are
    # shared by all 74 workers, 57 or 58 each.  A range that starts inside a tile contributes to it (first
    # item of its worker); a range that starts a tile owns it (last item).
    tiles, workers, nkb = 96, 74, 192
    owners, contributors = {}, {}
    for w in range(workers):
        items = B.exo_gemm_schedule_work(tiles, workers, workers, nkb, w)
        whole = [(k, it) for k, it in enumerate(items) if it[2] == 1]
        assert [it[0] for _, it in whole] == [w]                       # its tile of the whole wave
        for k, (tile, sl, n_sl, b, e) in enumerate(items):
            if n_sl == 1:
                continue
            assert tile >= workers
            if sl == 0:
                assert b == 0 and k > whole[0][0] and k == len(items) - 1
                owners[tile] = w
            else:
                assert b > 0 and k < whole[0][0]
                contributors.setdefault(tile, []).append((sl, w))
    assert sorted(owners) == list(range(74, 96))
    for tile, own in owners.items():
        cs = sorted(contributors[tile])
        assert [sl for sl, _ in cs] == list(range(1, len(cs) + 1))
        assert [w for _, w in cs] == [own + k for k in range(1, len(cs) + 1)]   # consecutive workers, in K order
        assert 3 <= len(cs) + 1 <= 5                                           # 74 / 22 = 3.4 workers per tile


def test_whole_slices_keep_owners_and_contributors_in_groups():
    # 256 tiles on 74 workers, the 34 tail tiles cut in two whole slices: workers 0..33 own a tail tile and
    # compute their slice after their whole tiles; workers 34..67 contribute and compute theirs before; the
    # rest have none.  With an owner_extra of 3 the owning slice is 3 k-blocks longer.
    tiles, workers, nkb = 256, 74, 64
    full = (tiles // workers) * workers
    for extra in (0, 3):
        for w in range(workers):
            items = B.exo_gemm_schedule_work(tiles, workers, 68, nkb, w, owner_extra=extra)
            unit = [k for k, it in enumerate(items) if it[0] >= full]
            if w < 34:
                assert unit == [len(items) - 1] and items[-1] == (full + w, 0, 2, 0, 32 + extra)
            elif w < 68:
                assert unit == [0] and items[0] == (full + w - 34, 1, 2, 32 + extra, 64)
            else:
                assert unit == []
            assert [it[0] for it in items if it[0] < full] == [w + k * workers for k in range(3)]


def test_work_schedule_rejects_impossible_plans():
    with pytest.raises(ValueError):
        B.exo_gemm_schedule_work(256, 74, 20, 64, 0)       # fewer sharing workers than the 34 tail tiles
    with pytest.raises(ValueError):
        B.exo_gemm_schedule_work(256, 74, 75, 64, 0)       # more than there are workers
    with pytest.raises(ValueError):
        B.exo_gemm_schedule_work(149, 148, 8, 4, 0)        # one tail tile of 4 k-blocks cannot feed 8 workers
    with pytest.raises(ValueError):
        B.exo_gemm_schedule_work(148, 148, 8, 64, 0)       # no tail to share


def test_plan_preview_shares_the_partial_last_wave():
    # 4096^3 with 256x256 pair tiles: 256 tiles on 74 pairs = 3 whole waves + 34 tiles, each cut in two
    # whole slices (68 of the 74 pairs take one)
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, c_dtype=B.BF16), 148)
    i = info.as_dict()
    assert (i["cta_group"], i["tile_n"]) == (2, 256) and i["tail_tiles"] == 34
    assert i["tail_workers"] == 68 and i["split_k"] == 2
    assert i["workspace_bytes"] == 34 * 1 * 256 * 256 * 4
    # never cut when told not to, and never more slices than fit the workers or the K loop
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, flags=B.flag_split_k(1)), 148)
    assert info.split_k == 1 and info.workspace_bytes == 0 and info.tail_workers == 0
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, flags=B.flag_split_k(2)), 148)
    assert info.tail_workers == 68 and info.split_k == 2
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=256), 148)
    assert info.split_k == 1                           # 256 k-elements: nothing to cut
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=12288), 148)
    i = info.as_dict()
    assert i["split_k"] >= 2 and i["tail_tiles"] <= i["tail_workers"] <= i["grid"] // i["cta_group"]
    # a wave count that whole slices cannot fix: 48 tiles of 256 x 256 on 74 pairs.  No two slices per tile fit,
    # so the 48 x 192 k-blocks are shared out among all 74 pairs in equal ranges that ignore tile boundaries
    st, info = B.exo_gemm_plan_preview(good(M=1000, N=3072, K=12288, flags=B.flag_cta_group(2) | B.flag_tile_n(256)), 148)
    i = info.as_dict()
    assert i["tail_tiles"] == 48 and i["tail_workers"] == 74 and i["split_k"] in (2, 3)
    assert B.exo_gemm_validate(good(flags=B.flag_split_k(9))) == B.ERR_INVALID_ARG


def test_batched_create_checks_its_arguments_before_touching_cuda():
    d = good(M=256, N=192, K=128)                       # C row-major fp32, ldc = 192: one C spans 256*192 elements
    c_extent = 255 * 192 + 192
    assert B.exo_gemm_create_batched(d, 0, 0, 0, c_extent)[0] == B.ERR_INVALID_ARG          # batch_count < 1
    assert B.exo_gemm_create_batched(d, 70000, 0, 0, c_extent)[0] == B.ERR_INVALID_ARG
    assert B.exo_gemm_create_batched(d, 4, -8, 0, c_extent)[0] == B.ERR_INVALID_ARG
    assert B.exo_gemm_create_batched(d, 4, 256 * 128, 192 * 128, c_extent - 4)[0] == B.ERR_INVALID_ARG   # C overlap
    assert B.exo_gemm_create_batched(d, 4, 256 * 128 + 4, 192 * 128, c_extent)[0] == B.ERR_UNSUPPORTED   # 8 bytes off
    assert B.exo_gemm_create_batched(d, 4, 256 * 128, 192 * 128, c_extent + 2)[0] == B.ERR_UNSUPPORTED
    import torch
    if not torch.cuda.is_available():                   # well-formed: only the missing GPU stops it
        assert B.exo_gemm_create_batched(d, 4, 256 * 128, 0, c_extent)[0] in (B.ERR_CUDA, B.ERR_ARCH)


def test_shared_operand_cluster_flags_and_preview():
    ALWAYS, SUBST = B.FLAG2_SHARE_ALWAYS, B.FLAG2_SHARE_SUBSTITUTED
    assert B.exo_gemm_validate(good(flags2=B.FLAG2_SHARE_NEVER)) == B.OK
    for f2 in (ALWAYS, SUBST):
        assert B.exo_gemm_validate(good(flags2=f2)) == B.OK
        assert B.exo_gemm_validate(good(flags2=f2, flags=B.flag_cta_group(1))) == B.ERR_INVALID_ARG
        assert B.exo_gemm_validate(good(flags2=f2, flags=B.flag_tile_n(128))) == B.ERR_INVALID_ARG
        assert B.exo_gemm_validate(good(flags2=f2, flags=B.flag_grid_limit(6))) == B.ERR_INVALID_ARG
        assert B.exo_gemm_validate(good(flags2=f2, flags=B.flag_grid_limit(8) | B.flag_tile_n(256))) == B.OK
    assert B.exo_gemm_validate(good(flags2=64)) == B.ERR_INVALID_ARG
    have = B.exo_gemm_has_shared_operand_clusters()
    assert have in (0, 1)
    st, info = B.exo_gemm_plan_preview(good(M=8192, N=8192, K=8192, flags2=ALWAYS), 148)
    if not have:
        assert st == B.ERR_UNSUPPORTED
        return
    i = info.as_dict()
    # slots of four CTAs, each covering 256 x 512 of C per step; 148 SMs hold 37 of them
    assert st == B.OK and (i["cluster_size"], i["cta_group"], i["tile_m"], i["tile_n"]) == (4, 2, 256, 256)
    assert (i["tiles_m"], i["tiles_n"], i["grid"]) == (32, 16, 148)
    assert i["tail_tiles"] == 512 % 37 and (i["tail_workers"] == 0 or i["tail_tiles"] < i["tail_workers"] <= 37)
    # the K-slices' scratch covers both tiles of a slot
    assert i["workspace_bytes"] == i["tail_tiles"] * (i["split_k"] - 1) * 2 * 256 * 256 * 4
    st, info = B.exo_gemm_plan_preview(good(M=600, N=700, K=64, flags2=SUBST, flags=B.flag_grid_limit(4)), 148)
    assert st == B.OK and (info.cluster_size, info.grid, info.tiles_m, info.tiles_n) == (4, 4, 3, 2)
    # left to itself the library keeps independent pairs, and a plain plan reports its CTA group as the cluster
    st, info = B.exo_gemm_plan_preview(good(M=8192, N=8192, K=8192), 148)
    assert st == B.OK and info.cluster_size == info.cta_group == 2


def test_base_library_has_no_shared_operand_kernels():
    import ctypes
    from paper_2609_16389_b200 import build as cuda_build
    base = ctypes.CDLL(cuda_build.build())
    base.exo_gemm_has_shared_operand_clusters.restype = ctypes.c_int32
    assert base.exo_gemm_has_shared_operand_clusters() == 0
    base.exo_gemm_plan_preview.argtypes = [ctypes.POINTER(B.Desc), ctypes.c_int32, ctypes.POINTER(B.Info)]
    info = B.Info()
    d = good(M=1024, N=1024, K=1024, flags2=B.FLAG2_SHARE_ALWAYS)
    assert base.exo_gemm_plan_preview(ctypes.byref(d), 148, ctypes.byref(info)) == B.ERR_UNSUPPORTED
    d = good(M=1024, N=1024, K=1024)
    assert base.exo_gemm_plan_preview(ctypes.byref(d), 148, ctypes.byref(info)) == B.OK and info.cluster_size == info.cta_group
    for name in B.EXPORTED_SYMBOLS:
        getattr(base, name)


def test_tall_tile_flags_and_preview():
    TALL, REG = B.flag2_cta_rows(256), B.flag2_cta_rows(128)
    assert (TALL, REG) == (8, 4)
    assert B.exo_gemm_validate(good(flags2=TALL)) == B.OK and B.exo_gemm_validate(good(flags2=REG)) == B.OK
    assert B.exo_gemm_validate(good(flags2=12)) == B.ERR_INVALID_ARG                      # rows field 3
    assert B.exo_gemm_validate(good(flags2=TALL, flags=B.flag_cta_group(1))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags2=TALL, flags=B.flag_tile_n(128))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags2=TALL, flags=B.flag_k_subblocks(2))) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags2=TALL | B.FLAG2_SHARE_ALWAYS)) == B.ERR_INVALID_ARG
    assert B.exo_gemm_validate(good(flags2=TALL | B.FLAG2_SHARE_NEVER)) == B.OK
    st, info = B.exo_gemm_plan_preview(good(M=1000, N=520, K=264, flags2=TALL), 148)
    i = info.as_dict()
    assert st == B.OK and (i["cta_group"], i["tile_m"], i["tile_n"], i["tile_k"]) == (2, 512, 256, 64)
    assert (i["tiles_m"], i["tiles_n"], i["grid"], i["tmem_columns"]) == (2, 3, 12, 512)
    # a stage holds 256 rows of A and this CTA's 128 rows of B
    assert i["stages"] * 49152 + 32768 * i["epilogue_buffers"] + 1536 == i["smem_bytes"] <= 232448
    # a long K loop amortises the exposed epilogue: such problems take the tall tile on their own where it fills
    # the waves as well as the 128-row tile does; 4096^3 (two uneven waves of 512 x 256 tiles) does not
    st, info = B.exo_gemm_plan_preview(good(M=4608, N=4096, K=16384, c_dtype=B.BF16), 148)
    assert info.tile_m == 512 and info.stages == 4 and info.split_k == 1
    st, info = B.exo_gemm_plan_preview(good(M=4096, N=4096, K=4096, c_dtype=B.BF16), 148)
    assert info.tile_m == 256
    st, info = B.exo_gemm_plan_preview(good(M=8192, N=8192, K=8192, flags2=REG), 148)
    assert info.tile_m == 256
    # the K-slices' scratch covers both accumulators of both CTAs
    st, info = B.exo_gemm_plan_preview(good(M=2560, N=3840, K=2048, flags2=TALL), 148)
    assert (info.tail_tiles, info.split_k, info.workspace_bytes) == (1, 2, 1 * 512 * 256 * 4)   # slices of 1024 k
    st, info = B.exo_gemm_plan_preview(good(M=2560, N=3840, K=2048, flags2=TALL, flags=B.flag_split_k(8)), 148)
    assert (info.tail_tiles, info.split_k, info.workspace_bytes) == (1, 8, 7 * 512 * 256 * 4)   # on request: 256 k


def test_lean_kernel_flags_and_preview():
    LEAN, NEVER = B.FLAG2_LEAN_ALWAYS, B.FLAG2_LEAN_NEVER
    assert (LEAN, NEVER) == (32, 16)
    assert B.exo_gemm_validate(good(flags2=LEAN)) == B.OK and B.exo_gemm_validate(good(flags2=NEVER)) == B.OK
    assert B.exo_gemm_validate(good(flags2=48)) == B.ERR_INVALID_ARG                       # lean field 3
    assert B.exo_gemm_validate(good(flags2=64)) == B.ERR_INVALID_ARG                       # bits 6.. are reserved
    for f, f2 in [(B.flag_cta_group(2) | B.flag_split_k(2), LEAN), (B.flag_tile_n(256), LEAN), (B.flag_split_k(3), LEAN), (B.flag_split_k(8), LEAN),
                  (B.flag_grid_limit(8), LEAN), (1 << 11, LEAN), (0, LEAN | B.flag2_cta_rows(256)),
                  (0, LEAN | B.FLAG2_SHARE_ALWAYS)]:
        assert B.exo_gemm_validate(good(flags=f, flags2=f2)) == B.ERR_INVALID_ARG, (f, f2)
    assert B.exo_gemm_validate(good(flags=B.flag_split_k(1) | B.flag_tile_n(128), flags2=LEAN | B.FLAG2_SHARE_NEVER)) == B.OK
    # 128 x 64 tiles while a CTA per tile fits the SMs, else 128 x 128; a ring no deeper than the K loop
    st, info = B.exo_gemm_plan_preview(good(M=256, N=256, K=256, flags2=LEAN), 148)
    i = info.as_dict()
    assert st == B.OK and (i["lean_kernel"], i["cta_group"], i["tile_m"], i["tile_n"], i["tile_k"]) == (1, 1, 128, 64, 128)
    assert (i["tiles_m"], i["tiles_n"], i["grid"], i["stages"], i["tmem_columns"], i["split_k"]) == (2, 4, 8, 2, 64, 1)
    # fp32 C: two 4 KB staging buffers per TMEM lane quadrant; a stage holds 128 rows of A and 64 of B, 128 k each
    assert i["smem_bytes"] == 2 * 49152 + 8 * 4096 + 512 + 1024
    st, info = B.exo_gemm_plan_preview(good(M=1024, N=1024, K=4096, c_dtype=B.BF16, flags2=LEAN), 148)
    i = info.as_dict()
    assert (i["lean_kernel"], i["tile_n"], i["grid"], i["stages"]) == (1, 64, 128, 4) and i["smem_bytes"] <= 232448
    st, info = B.exo_gemm_plan_preview(good(M=1024, N=2048, K=512, flags2=LEAN), 148)
    assert (info.lean_kernel, info.tile_n, info.grid, info.stages) == (1, 128, 128, 2)      # 64 KB of staging for an fp32 C
    st, info = B.exo_gemm_plan_preview(good(M=1024, N=2048, K=512, flags2=LEAN, flags=B.flag_tile_n(64)), 148)
    assert (info.lean_kernel, info.tile_n, info.grid) == (1, 64, 256)                      # more CTAs than SMs: they queue
    st, info = B.exo_gemm_plan_preview(good(M=1024, N=2048, K=512, flags2=NEVER), 148)
    assert info.lean_kernel == 0
    # the library's own choice: one wave of 128 x 64 tiles up to K = 2048, a cluster per tile from K ~ 1000 on where
    # the SMs have room for it, 128 x 128 tiles at K = 512 only; never when the caller names a persistent-kernel parameter
    for (M, N, K), want in {(256, 256, 256): (1, 64, 1, 8), (512, 512, 512): (1, 64, 1, 32), (512, 512, 2048): (1, 64, 4, 128),
                            (512, 1000, 3072): (1, 64, 2, 128), (1000, 1000, 1000): (1, 64, 1, 128), (512, 1000, 6144): (0,),
                            (1000, 1000, 3072): (0,), (512, 3072, 512): (1, 128, 1, 96), (512, 3072, 1000): (0,),
                            (2048, 2048, 512): (0,), (4096, 4096, 4096): (0,)}.items():
        st, info = B.exo_gemm_plan_preview(good(M=M, N=N, K=K), 148)
        got = (info.lean_kernel, info.tile_n, info.split_k, info.grid) if info.lean_kernel else (0,)
        assert st == B.OK and got == want, (M, N, K, got)
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=2048, flags=B.flag_split_k(1)), 148)
    assert (info.lean_kernel, info.split_k, info.grid) == (1, 1, 32)                    # "never cut K" is kept
    for f in (B.flag_tile_n(64), B.flag_cta_group(1), B.flag_max_stages(3), B.flag_epi_buffers(1), B.flag_band(2), B.flag_split_k(4)):
        st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=512, flags=f), 148)
        assert info.lean_kernel == 0, f
    # a CTA pair per 256 x 256 (or 256 x 128) tile on request
    st, info = B.exo_gemm_plan_preview(good(M=2048, N=2048, K=512, flags2=LEAN, flags=B.flag_cta_group(2)), 148)
    i = info.as_dict()
    assert (i["lean_kernel"], i["cta_group"], i["tile_m"], i["tile_n"], i["cluster_size"], i["grid"], i["stages"], i["tmem_columns"]) == (1, 2, 256, 256, 2, 128, 7, 256)
    assert i["smem_bytes"] == 7 * 32768 + 512 + 1024
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=128, flags2=LEAN, flags=B.flag_cta_group(2) | B.flag_tile_n(128)), 148)
    assert (info.tile_n, info.stages, info.grid, info.smem_bytes) == (128, 1, 16, 128 * 128 * 4 + 512 + 1024)   # the ring holds the staged C
    # K cut over a cluster of 2 or 4 CTAs per tile; the partial sums travel through shared memory, not a workspace
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=1000, flags2=LEAN, flags=B.flag_split_k(4)), 148)
    i = info.as_dict()
    assert (i["lean_kernel"], i["split_k"], i["cluster_size"], i["grid"], i["stages"], i["workspace_bytes"]) == (1, 4, 4, 128, 2, 0)
    assert i["smem_bytes"] == 2 * 49152 + 8 * 4096 + 3 * 2 * 4096 + 512 + 1024         # + three peers' 32 x 64 fp32 parts
    st, info = B.exo_gemm_plan_preview(good(M=512, N=512, K=128, flags2=LEAN, flags=B.flag_split_k(4)), 148)
    assert (info.split_k, info.cluster_size, info.grid) == (1, 1, 32)                   # one k-block: nothing to cut


def test_smoke_cases_are_in_the_supported_set():
    import __graft_entry__ as entry
    from paper_2609_16389_b200 import harness
    for p in entry.smoke_cases():
        d = harness.desc_of(p)
        assert B.exo_gemm_validate(d) == B.OK, p.name
        assert B.exo_gemm_plan_preview(d, 148)[0] == B.OK, p.name
