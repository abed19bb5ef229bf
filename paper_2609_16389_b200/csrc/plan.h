// Host-side planning: argument validation, canonical form, tile-shape choice.
// Pure functions (no CUDA calls), so they can be exercised without a GPU.
#pragma once
#include <math.h>
#include <stdint.h>

#include "../../include/exo_gemm.h"
#include "gemm_params.h"

namespace exo {

inline int elem_bytes(int dtype) { return dtype == EXO_GEMM_FP32 ? 4 : 2; }

struct FlagOverrides {
  int split;       // 0 = auto, 1 = never split, 2..8 = slices per tail tile (if they fit)
  bool no_workspace;  // set by the allocation-free entry point: nothing that needs device scratch
  bool reduce_add;    // the parts of a cut tile meet in C by TMA reduce-add instead of in a workspace
  int epi_bufs;    // 0 = auto
  int stages;      // 0 = as many as fit, else an upper limit
  int ksub;        // 0 = auto
  int cta_group;   // 0 = auto
  int tile_n;      // 0 = auto
  int band;        // 0 = auto
  int along_m;     // 0 = auto/default, 1 = forced
  int grid_limit;  // 0 = none
  int share;       // clusters of two CTA pairs sharing the loads of A: 0 = auto, 1 = never, 2 = always,
                   // 3 = always, but every slot launched as two plain pairs (exercises the substitute path)
  int mrep;        // 128-row blocks of C per CTA: 0 = auto, 1, or 2 (the tall 2-CTA tile, 512 x 256 per pair)
  int lean;        // the one-tile-per-CTA kernel for problems of less than one wave: 0 = auto, 1 = never, 2 = always
};

inline FlagOverrides decode_flags(uint32_t f, uint32_t f2 = 0) {
  FlagOverrides o;
  o.cta_group = (int)(f & 3u);
  o.tile_n = (int)((f >> 2) & 15u) * 64;
  o.band = (int)((f >> 6) & 15u);
  o.along_m = (int)((f >> 10) & 1u);
  o.grid_limit = (int)((f >> 12) & 255u);
  o.ksub = (int)((f >> 20) & 3u);
  o.epi_bufs = (int)((f >> 22) & 3u);
  o.stages = (int)((f >> 24) & 15u);
  o.split = (int)((f >> 28) & 15u);
  o.no_workspace = false;
  o.reduce_add = (f & (1u << 11)) != 0;
  o.share = (int)(f2 & 3u);
  o.mrep = (int)((f2 >> 2) & 3u);
  o.lean = (int)((f2 >> 4) & 3u);
  return o;
}

inline exo_gemm_status_t validate_desc(const exo_gemm_desc_t* d) {
  if (!d) return EXO_GEMM_ERR_NULL;
  if ((d->flags2 & ~63u) != 0 || ((d->flags2 >> 2) & 3u) == 3u || ((d->flags2 >> 4) & 3u) == 3u) return EXO_GEMM_ERR_INVALID_ARG;
  const int64_t kMaxDim = 2147483647LL;
  if (d->M < 0 || d->N < 0 || d->K < 0 || d->M > kMaxDim || d->N > kMaxDim || d->K > kMaxDim)
    return EXO_GEMM_ERR_INVALID_ARG;
  auto bad_dtype = [](int32_t t) { return t < EXO_GEMM_BF16 || t > EXO_GEMM_FP32; };
  auto bad_layout = [](int32_t l) { return l != EXO_GEMM_ROW_MAJOR && l != EXO_GEMM_COL_MAJOR; };
  if (bad_dtype(d->ab_dtype) || bad_dtype(d->c_dtype)) return EXO_GEMM_ERR_INVALID_ARG;
  if (bad_layout(d->a_layout) || bad_layout(d->b_layout) || bad_layout(d->c_layout))
    return EXO_GEMM_ERR_INVALID_ARG;
  if (d->device < -1) return EXO_GEMM_ERR_INVALID_ARG;
  auto extent = [](int32_t layout, int64_t rows, int64_t cols) {
    const int64_t e = layout == EXO_GEMM_ROW_MAJOR ? cols : rows;
    return e < 1 ? 1 : e;
  };
  const int64_t kMaxLd = (1LL << 36);
  if (d->lda < extent(d->a_layout, d->M, d->K) || d->ldb < extent(d->b_layout, d->K, d->N) ||
      d->ldc < extent(d->c_layout, d->M, d->N) || d->lda > kMaxLd || d->ldb > kMaxLd || d->ldc > kMaxLd)
    return EXO_GEMM_ERR_INVALID_ARG;
  if (((d->flags >> 28) & 15u) > 8u) return EXO_GEMM_ERR_INVALID_ARG;
  if (((d->flags >> 20) & 3u) == 3u || ((d->flags >> 22) & 3u) == 3u) return EXO_GEMM_ERR_INVALID_ARG;
  if (((d->flags >> 24) & 15u) == 1u || ((d->flags >> 24) & 15u) > (uint32_t)kMaxStages) return EXO_GEMM_ERR_INVALID_ARG;
  const FlagOverrides o = decode_flags(d->flags, d->flags2);
  if (o.cta_group == 3) return EXO_GEMM_ERR_INVALID_ARG;
  if (o.tile_n != 0 && o.tile_n != 64 && o.tile_n != 128 && o.tile_n != 256) return EXO_GEMM_ERR_INVALID_ARG;
  if (o.cta_group == 2 && o.tile_n == 64) return EXO_GEMM_ERR_INVALID_ARG;
  if (o.grid_limit != 0 && o.cta_group == 2 && (o.grid_limit & 1)) return EXO_GEMM_ERR_INVALID_ARG;
  // forcing the shared-operand clusters fixes the tile shape they are built for
  if (o.share >= 2 && (o.cta_group == 1 || (o.tile_n != 0 && o.tile_n != 256) || (o.grid_limit & 3)))
    return EXO_GEMM_ERR_INVALID_ARG;
  // so does forcing the tall tile, which has no shared-operand form
  if (o.mrep == 2 && (o.cta_group == 1 || (o.tile_n != 0 && o.tile_n != 256) || o.ksub == 2 || o.share >= 2))
    return EXO_GEMM_ERR_INVALID_ARG;
  // the reduce-add form of the K split exists for plain tiles only
  if ((d->flags & (1u << 11)) && (o.share >= 2 || o.mrep == 2)) return EXO_GEMM_ERR_INVALID_ARG;
  // the one-tile-per-CTA kernel has 1-CTA tiles of 128 x 64 or 128 x 128, cuts K over a cluster of 2 or 4 only and
  // takes every tile at once
  // (with CTA_GROUP(2): one 256 x 128 or 256 x 256 tile per CTA pair, K never cut)
  if (o.lean == 2 && (o.share >= 2 || o.mrep == 2 || (d->flags & (1u << 11)) || o.grid_limit != 0 ||
                      (o.cta_group == 2 ? o.split >= 2 : (o.tile_n == 256 || (o.split >= 2 && o.split != 2 && o.split != 4)))))
    return EXO_GEMM_ERR_INVALID_ARG;
  // beyond here the call is a legal BLAS call; what follows is this library's supported set
  // fp32 operands are multiplied as tf32 (the precision of the paper's own kernels) into an fp32 C
  if (d->c_dtype != EXO_GEMM_FP32 && d->c_dtype != d->ab_dtype) return EXO_GEMM_ERR_UNSUPPORTED;
  // the reduce-add form of the K split adds fp32 partial sums onto an fp32 C
  if ((d->flags & (1u << 11)) && d->c_dtype != EXO_GEMM_FP32) return EXO_GEMM_ERR_UNSUPPORTED;
  // the persistent scheduler indexes tiles (at least 128 x 64 each) and k-blocks with 32 bits
  if (((d->M + 127) / 128) * ((d->N + 63) / 64) >= (1LL << 31)) return EXO_GEMM_ERR_UNSUPPORTED;
  // (a leading dimension whose byte size is not a multiple of 16 cannot be described by a tensor map: a plan
  // repacks such a matrix through scratch of its own, see repack_mask; the entry points that own no scratch refuse it)
  return EXO_GEMM_OK;
}

// Which matrices (1 = A, 2 = B, 4 = C) have rows that do not start on 16-byte boundaries and have to go through
// an aligned copy.  A matrix that is never touched (empty problem, K == 0) has no stride rule.
inline int repack_mask(const exo_gemm_desc_t& d) {
  const bool c_used = d.M > 0 && d.N > 0;
  const bool ab_used = c_used && d.K > 0;
  int m = 0;
  if (ab_used && (d.lda * elem_bytes(d.ab_dtype)) % 16) m |= 1;
  if (ab_used && (d.ldb * elem_bytes(d.ab_dtype)) % 16) m |= 2;
  if (c_used && (d.ldc * elem_bytes(d.c_dtype)) % 16) m |= 4;
  return m;
}

// Rows (outer) and contiguous elements per row (inner) of a matrix as it lies in memory.
inline void storage_shape(int32_t layout, int64_t rows, int64_t cols, int64_t* outer, int64_t* inner) {
  *outer = layout == EXO_GEMM_ROW_MAJOR ? rows : cols;
  *inner = layout == EXO_GEMM_ROW_MAJOR ? cols : rows;
}

// Strided batch: `batch` matrices, consecutive ones stride_x elements apart.  A and B may repeat
// (stride 0); C matrices must not overlap.  Strides obey the same 16-byte rule as leading dimensions.
inline exo_gemm_status_t validate_batch(const exo_gemm_desc_t* d, int64_t batch, int64_t sa, int64_t sb, int64_t sc) {
  exo_gemm_status_t st = validate_desc(d);
  if (st != EXO_GEMM_OK) return st;
  if (batch < 1 || batch > 65535 || sa < 0 || sb < 0 || sc < 0) return EXO_GEMM_ERR_INVALID_ARG;
  const int64_t kMaxStride = 1LL << 38;
  if (sa > kMaxStride || sb > kMaxStride || sc > kMaxStride) return EXO_GEMM_ERR_INVALID_ARG;
  if (batch > 1) {
    if (repack_mask(*d)) return EXO_GEMM_ERR_UNSUPPORTED;   // the repacking path has no strided-batch form
    const int64_t c_extent = d->c_layout == EXO_GEMM_ROW_MAJOR ? (d->M - 1) * d->ldc + d->N : (d->N - 1) * d->ldc + d->M;
    if (d->M > 0 && d->N > 0 && sc < c_extent) return EXO_GEMM_ERR_INVALID_ARG;  // overlapping outputs
    if ((sa * elem_bytes(d->ab_dtype)) % 16 || (sb * elem_bytes(d->ab_dtype)) % 16 ||
        (sc * elem_bytes(d->c_dtype)) % 16)
      return EXO_GEMM_ERR_UNSUPPORTED;
    if (((d->M + 127) / 128) * ((d->N + 63) / 64) * batch >= (1LL << 31)) return EXO_GEMM_ERR_UNSUPPORTED;
  }
  return EXO_GEMM_OK;
}

// The problem after canonicalisation: C is always written row-major.  A
// column-major C is computed as C^T = B^T A^T, which only swaps the operands and
// M with N; an operand's "major-ness" (is K or M/N contiguous) carries over.
struct Canonical {
  int64_t M, N, K;
  int a_mn_major, b_mn_major;  // of the canonical operands
  int64_t lda, ldb, ldc;
  int swapped;
  int ab_bytes;                          // 2 (bf16/fp16) or 4 (fp32 storage, tf32 math)
  int c_bytes;                           // 2 or 4: element size of C
  int64_t batch;                         // matrices in a strided batch (1 = plain GEMM)
  int64_t stride_a, stride_b, stride_c;  // elements between consecutive matrices (canonical operands)
};

inline Canonical canonicalize(const exo_gemm_desc_t& d, int64_t batch = 1, int64_t stride_a = 0,
                              int64_t stride_b = 0, int64_t stride_c = 0) {
  Canonical c;
  c.ab_bytes = elem_bytes(d.ab_dtype);
  c.c_bytes = elem_bytes(d.c_dtype);
  c.batch = batch;
  c.stride_c = stride_c;
  c.stride_a = d.c_layout == EXO_GEMM_COL_MAJOR ? stride_b : stride_a;
  c.stride_b = d.c_layout == EXO_GEMM_COL_MAJOR ? stride_a : stride_b;
  const int a_mn = d.a_layout == EXO_GEMM_COL_MAJOR;  // A (M x K) col-major: M contiguous
  const int b_mn = d.b_layout == EXO_GEMM_ROW_MAJOR;  // B (K x N) row-major: N contiguous
  c.swapped = d.c_layout == EXO_GEMM_COL_MAJOR;
  c.K = d.K;
  c.ldc = d.ldc;
  if (!c.swapped) {
    c.M = d.M; c.N = d.N;
    c.a_mn_major = a_mn; c.b_mn_major = b_mn;
    c.lda = d.lda; c.ldb = d.ldb;
  } else {
    c.M = d.N; c.N = d.M;
    c.a_mn_major = b_mn; c.b_mn_major = a_mn;
    c.lda = d.ldb; c.ldb = d.lda;
  }
  return c;
}

struct TileConfig {
  int64_t full_tiles;      // tiles dealt round-robin as whole-K work items (whole waves)
  int tail_tiles;          // the tiles of the partial last wave
  int tail_workers;        // workers that share those tiles' k-blocks in equal consecutive ranges (0: not cut)
  int split;               // the most K-slices any tail tile is cut into (1: not cut) = slots + 1
  int slots;               // partial-sum slots per tail tile in the workspace
  int snap;                // range boundaries this close to a tile boundary (k-blocks) are moved onto it
  int owner_extra;         // whole slices side by side: k-blocks the owning slice takes beyond an even share
  int64_t workspace_bytes; // fp32 partials of the contributing slices of the tail tiles
  int cta_group, tile_n, ksub, stages, epi_bufs;
  int stages_direct;       // ring depth of a run that stores C straight from registers (no staging buffers);
                           // 0: this plan always stages (a staging depth was requested)
  int pairs;               // CTA pairs per cluster (2: the pairs share the loads of A; else 1)
  int mrep;                // 128-row blocks of C per CTA (2: the tall tile; else 1)
  int tiles_m, tiles_n;    // tiles of (128 * cta_group) x (tile_n * pairs): what one cluster computes at a time
  int band, along_m;
  int workers;  // CTA groups launched
  int lean;     // > 0: the one-tile-per-CTA kernel runs this plan (workers = tiles, `stages` is its ring) with clusters of
                // this many CTAs (1, 2 or 4) sharing each tile's K loop
};

// Sub-blocks of 64 k-elements per pipeline stage.  Two per stage halves the number of
// barrier round trips per MMA, which is what bounds the issuing thread when a tile's
// MMAs are short (N <= 128); with N = 256 on one CTA two would leave only two stages.
inline int default_ksub(int cta_group, int bn) { (void)cta_group; return bn == 256 ? 1 : 2; }

// Main-loop throughput of a tile shape relative to the 2-CTA 256x256 tile, measured on
// a B200 at 4096^3 with the wave-quantisation factor divided out: smaller N per CTA
// moves more operand bytes through shared memory per flop and leaves the issuing
// thread less time per MMA.
inline double shape_efficiency(int cta_group, int bn) {
  if (cta_group == 2) return bn == 256 ? 1.0 : 0.81;
  return bn == 256 ? 0.86 : (bn == 128 ? 0.66 : 0.40);
}

// Main-loop speed of the shared-operand clusters relative to independent pairs.  With operand rows that
// start on 128-byte boundaries the halved fetches of A do not show as time; with rows that do not
// (K = 1000 16-bit elements: 2000 bytes) every 128-byte piece of a box straddles two lines, the L2 sees
// twice the requests, and fetching less pays: +0.2 to +10 %, typically +1.5 %, over the 24 sweep shapes
// with K = 1000 that take 256 x 256 tiles (never slower).
constexpr double kShareGain = 1.0;
constexpr double kShareGainUnalignedRows = 1.02;
// Main-loop speed of the tall tile (256 rows per CTA) relative to the 128-row tile, and the clocks
// per tile its exposed epilogue costs.
constexpr double kTallGain = 1.06;
constexpr double kTallDrain = 4000.0;

// k-elements in one 128-byte sub-block row: 64 for 16-bit operands, 32 for fp32 storage.
inline int sub_block_k(int ab_bytes) { return 128 / ab_bytes; }

// A part of a tail tile shorter than this many k-blocks is not worth the exchange of its partial sums
// (reading one back costs the owner about 16 * tile_n clocks, a k-block takes 2 * tile_n * ksub).
inline int32_t tail_snap(int ksub) { return 8 / ksub; }

// How many workers share the k-blocks of the partial last wave's tiles (0 = those tiles stay whole).
// The tail's tail * num_k_blocks k-blocks are cut into that many equal consecutive ranges; a tile is then
// computed by tail_workers / tail workers on average and the last wave takes tail / tail_workers of a
// tile's time, plus the exchange of partial sums.
// (K is given in units of 128-byte sub-block rows x 64, i.e. already scaled by the element size.)
inline int tail_workers_for(int64_t tiles, int64_t workers, int64_t K, int ksub, const FlagOverrides& o, int mrep = 1) {
  const int64_t tail = tiles % workers;
  if (tail == 0 || o.split == 1 || o.no_workspace) return 0;
  // A short K loop leaves no main-loop time to save, and the exchange of partial sums (a round trip
  // through L2 plus the extra output traffic) costs about as much as a dozen k-blocks.
  // Behind whole waves the contributing slices run first and the exchange is off the critical path
  // except for the owner's reading.  Measured there (one whole wave + 22 tiles of 256 x 256 on 74 pairs,
  // against the uncut tiles): two slices -19 % at K = 512, +3 to +5 % at K = 1000 and 1536, +7 to +8 % at
  // 2048, +8 to +10 % at 4096; three slices 0 %, -1 to -4 %, +4 to +5 %, +7 to +9 %: a further slice pays
  // only where it still keeps 2048 k-elements.
  // Problems smaller than one wave run all slices side by side and the owner waits for the others:
  // the split loses 28 % at K = 512 and 3 % at K = 1000, and wins 13-35 % from K = 2048 on.
  // (With three or more whole waves in front, the workers that start with a slice run out of step with
  // the rest for longer than the shorter last wave saves at K = 1024: -0.7 % at 4096 x 4096 x 1024.)
  const bool behind_waves = tiles >= workers;
  if (o.split == 0 && K < (behind_waves && tiles / workers <= 2 ? 960 : 2048)) return 0;
  const int64_t k_blocks = (K + kBlockK * ksub - 1) / (kBlockK * ksub);
  // slices per tile, on average: every slice keeps about 256 k-elements at least
  int64_t per_tile = (K / kBlockK) / 4;
  // (from K = 4096 on the owner finds the partials preloaded in its accumulator even behind a single whole
  // wave, and a third slice of 1365 k-elements wins another 2.7-4 % over two)
  if (o.split == 0 && behind_waves) per_tile = K >= 4096 ? K / 1365 : (K / 2048 > 2 ? K / 2048 : 2);
  if (per_tile > 8) per_tile = 8;
  if (o.split >= 2 && o.split < per_tile) per_tile = o.split;
  if (per_tile > k_blocks) per_tile = k_blocks;
  // Whole slices where at least two per tile fit the workers: every tail tile is cut at the same k-blocks
  // into f slices, one per worker (tail * f <= workers).
  const int64_t f = workers / tail < per_tile ? workers / tail : per_tile;
  if (f >= 2) return (int)(tail * f);
  if (per_tile < 2) return 0;
  // (not for the tall tile, whose partial sums are twice as large and whose epilogue nothing hides: 192 tiles
  // of 512 x 256 on 74 pairs at K = 12288 measured -8 %)
  if (mrep == 2 && o.split == 0) return 0;
  // More than half a wave of tail tiles: no two whole slices per tile fit, so the tail's k-blocks are shared
  // out among ALL workers in equal consecutive ranges that ignore tile boundaries (most tiles end up in
  // two parts).  Every worker then starts and ends with a part of a tile and exchanges partial sums, so
  // this pays only where the K loop is long and the last wave shrinks by a fifth of a tile or more
  // (measured against the uncut tiles: 48 tiles of 256 x 256 on 74 pairs at K = 12288 +4 %; 58 tiles behind
  // seven whole waves at K = 2048 -7 %).
  const int64_t tw = workers;
  // (Behind whole waves and with a very long K loop the tall tile is the better answer to such a tail: 192
  // tiles of 256 x 256 at K = 12288 measured 3-11 % slower in ranges than as 96 tall tiles.)
  if (o.split == 0 && behind_waves && K > 8192) return 0;
  if (o.split == 0) {
    // time saved against the exchange, both in clocks per column of the tile (a k-block of 64 takes 2;
    // a part's partial sums cost about 16 behind whole waves and about 38 side by side, as in
    // estimate_clocks): the saving has to be three times the exchange
    const double saved = (double)k_blocks * ksub * 2.0 * (1.0 - (double)tail / (double)tw);
    const double exchange = behind_waves ? 16.0 : 38.0;
    if (saved < 3.0 * exchange || tail * 5 > tw * 4) return 0;
  }
  return (int)tw;
}

// Estimated time of the whole problem in SM clocks for one candidate tile shape: whole waves of
// tiles, then the partial last wave (cut along K if that pays), plus what is exposed once per launch.
inline double estimate_clocks(int64_t M, int64_t N, int64_t K, int64_t batch, int cta_group, int bn,
                              int max_workers, const FlagOverrides& o, int pairs = 1, int mrep = 1,
                              bool mn_major_operand = false, bool unaligned_rows = false) {
  const int64_t tm = (M + 128 * cta_group * mrep - 1) / (128 * cta_group * mrep);
  const int64_t tn = (N + bn * pairs - 1) / (bn * pairs);
  const int64_t tiles = tm * tn * batch;
  if (tiles == 0) return 0.0;
  const int ksub = o.ksub ? o.ksub : (bn == 256 ? 1 : 2);
  const int64_t nkb = (K + kBlockK - 1) / kBlockK;
  double mainloop = (double)nkb * 2.0 * bn / shape_efficiency(cta_group, bn);  // clocks per whole tile
  if (pairs == 2) mainloop /= unaligned_rows ? kShareGainUnalignedRows : kShareGain;
  (void)mn_major_operand;  // M/N-contiguous operands run at the same rate (measured 1512 against 1516 TFLOP/s at 8192^3)
  // draining one accumulator: 5-7k clocks at N = 256, but only about a third less at N = 128 (waits, tile
  // decode and the last store's latency do not shrink with the tile: at K = 512 the 256-column tile is
  // 20-27 % faster than two 128-column ones)
  const double drain = 1500.0 + 16.0 * bn;
  // small K: the epilogue bounds a tile.  On top of either, about 2500 clocks per tile that neither hides
  // (measured: 23.7 against 21.7 us per 64-k-block tile at 4096^3; at K = 1000 one 256-column tile beats two
  // 128-column ones by 9-14 % where their main loops alone would tie)
  double per_tile = (mainloop > drain ? mainloop : drain) + 2500.0;
  if (mrep == 2) {  // two accumulators per tile, less operand traffic, but the epilogue is not hidden
    mainloop = 2.0 * mainloop / kTallGain;
    per_tile = mainloop + kTallDrain + 2.0 * 2500.0;   // it replaces two 128-row tiles and their fixed costs
  }
  const int64_t full_waves = tiles / max_workers;
  const int64_t tail = tiles % max_workers;
  double t = (double)full_waves * per_tile;
  if (tail > 0) {
    const int tw = tail_workers_for(tiles, max_workers, K, ksub, o, mrep);
    // a range of the tail + the exchange of partial sums (the tall tile's partials are twice as large and
    // nothing hides them).  Behind whole waves only the owner's reading of the partials is exposed (about
    // 4000 clocks per contributing slice of a 256-column tile); side by side, publishing and the round
    // trip are as well.
    if (tw > 0) {
      const int64_t parts = (tw + tail - 1) / tail;
      const double exchange = (full_waves > 0 ? 16.0 * (parts - 1) : 30.0 + 8.0 * (parts - 1)) * bn * mrep * mrep;
      // (ranges that ignore tile boundaries run about a sixth slower than their length says: tiles of one row or
      // column no longer fetch the same k-blocks at the same time, so fewer operand loads meet in L2.
      // Measured: 48 tiles on 74 pairs at K = 12288 gained 3-7 % where the ranges' length promised 35 %.)
      const double out_of_step = tw % tail != 0 ? 1.15 : 1.0;
      t += out_of_step * mainloop * (double)tail / (double)tw + 2500.0 + exchange;
    } else {
      t += per_tile;
    }
  }
  return t + drain + 3000.0;  // the last epilogue and the pipeline fill are exposed once
}

// Whether the one-tile-per-CTA kernel is the library's own choice, and with which tile width and how many
// CTAs per tile.  Measured against the persistent kernel's plan on every sweep shape of up to 300 tiles
// (launches replayed from CUDA graphs, bf16 and fp32 C): while 128 x 64 tiles fit the SMs at one CTA each it wins
// 12-30 % up to K = 2048; with room for two or four CTAs per tile a K loop from about 1000 on is cut over a
// cluster (512 x 512: +15 to +55 % up to K = 12288; 512 x 1000: +13 to +27 % up to K = 3072, level at 6144);
// 128 x 128 tiles win at K = 512 only (+18 to +26 %; +2 to +6 % at K = 1000); beyond one wave of those the
// persistent kernel's larger tiles are faster at every K.
inline bool lean_is_faster(const Canonical& c, const FlagOverrides& o, int sm_count, int* bn, int* split) {
  const int64_t k16 = c.K * (c.ab_bytes / 2);
  const int64_t t64 = ((c.M + 127) / 128) * ((c.N + 63) / 64), t128 = ((c.M + 127) / 128) * ((c.N + 127) / 128);
  *split = 1;
  if (k16 <= 0 || t128 <= 0) return false;
  if (t64 <= sm_count) {
    *bn = 64;
    if (k16 >= 960 && o.split == 0 && !o.no_workspace) *split = t64 * 4 <= sm_count ? 4 : (t64 * 2 <= sm_count ? 2 : 1);
    return k16 <= (*split == 4 ? 16384 : (*split == 2 ? 4096 : 2048));
  }
  if (t128 <= sm_count) {
    *bn = 128;
    return k16 <= 768;
  }
  return false;
}

inline TileConfig choose_config(const Canonical& c, const FlagOverrides& o, int sm_count,
                                int max_pairs /* co-resident 2-CTA clusters */,
                                int max_quads = 0 /* co-resident 4-CTA clusters; 0: variant not available */) {
  // (a plain local: a static here would be one process-wide object shared by every loaded build of the library)
  const int cand[7][4] = {{2, 256, 2, 1}, {2, 256, 1, 2}, {2, 256, 1, 1}, {2, 128, 1, 1},
                                 {1, 256, 1, 1}, {1, 128, 1, 1}, {1, 64, 1, 1}};
  int best_g = 0, best_n = 0, best_p = 1, best_r = 1;
  double best = 0;
  // operand rows (or columns, for M/N-contiguous storage) that do not start on 128-byte boundaries
  const bool unaligned_rows = c.K > 0 && (((c.lda * c.ab_bytes) % 128) != 0 || ((c.ldb * c.ab_bytes) % 128) != 0);
  for (int i = 0; i < 7; ++i) {
    const int g = cand[i][0], n = cand[i][1], pr = cand[i][2], mr = cand[i][3];
    if (mr == 2 && (o.mrep == 1 || o.share >= 2 || o.ksub == 2 || o.reduce_add)) continue;
    // The tall tile is the library's own choice only for problems of up to four waves of it: measured
    // against the 128-row tile it wins 2-6 % there at long K (6144^3, 6144 x 6144 x 12288, 4608 x 4096 x 16384)
    // and loses 2-5 % on larger problems (8192^3 with any C, 12288 x 6144 x 6144, 12288^3).
    if (mr == 2 && o.mrep == 0 && max_pairs >= 1 &&
        ((c.M + 511) / 512) * ((c.N + 255) / 256) * c.batch > 4 * (int64_t)max_pairs) continue;
    if (mr == 1 && o.mrep == 2 && max_pairs >= 1) continue;
    if (o.cta_group && o.cta_group != g) continue;
    if (o.tile_n && o.tile_n != n) continue;
    if (g == 2 && max_pairs < 1) continue;
    if (pr == 2 && (max_quads < 1 || o.share < 2)) continue;   // as a candidate only on request (but see below)
    if (pr == 1 && o.share >= 2 && max_quads >= 1) continue;
    const int workers = pr == 2 ? max_quads : (g == 2 ? max_pairs : sm_count);
    int w_eff = workers;
    if (o.grid_limit && o.grid_limit / (g * pr) < w_eff) w_eff = o.grid_limit / (g * pr);
    if (w_eff < 1) w_eff = 1;
    double t = estimate_clocks(c.M, c.N, c.K * (c.ab_bytes / 2), c.batch, g, n, w_eff, o, pr, mr,
                               c.a_mn_major || c.b_mn_major, unaligned_rows);
    if (mr == 2) t *= 1.03;  // the tall tile's exposed epilogue makes it the riskier choice: it must win clearly
    // candidates come largest tile first; a smaller one has to win by 3 %: the estimate flatters small tiles
    // (their fixed costs per tile are only partly modelled)
    if (best_g == 0 || t < best * 0.97) { best = t; best_g = g; best_n = n; best_p = pr; best_r = mr; }
  }
  if (best_g == 0) { best_g = o.cta_group ? o.cta_group : 1; best_n = o.tile_n ? o.tile_n : 128; }
  // Short K loops on one or two waves of 256 x 256 tiles: where 256 x 128 tiles fill their waves clearly
  // better they win (K = 512, 96 tiles of 256 x 256 on 74 pairs = 65 % against 192 on 222 = 86 %: +4 to +6 %
  // with a bf16 C, +0.4 to +2 % with an fp32 C), which the clock estimate above, made for many waves, does not
  // see; where both fill alike the wider tile stays (144 tiles: -8 to -14 % with 128 columns).
  if (best_g == 2 && best_n == 256 && best_p == 1 && best_r == 1 && max_pairs >= 1 && o.cta_group == 0 && o.tile_n == 0 &&
      o.mrep == 0 && o.share < 2 && o.grid_limit == 0 && c.K * (c.ab_bytes / 2) <= 512) {
    const int64_t t256 = ((c.M + 255) / 256) * ((c.N + 255) / 256) * c.batch;
    const int64_t t128 = ((c.M + 255) / 256) * ((c.N + 127) / 128) * c.batch;
    const int64_t w = max_pairs;
    const double fill256 = (double)t256 / (double)(((t256 + w - 1) / w) * w);
    const double fill128 = (double)t128 / (double)(((t128 + w - 1) / w) * w);
    if (t256 <= 2 * w && fill128 >= fill256 + 0.15) best_n = 128;
  }
  // Operand rows off the 128-byte grid at K around 1000 with a 16-bit C: the tall tile, which moves a quarter fewer
  // operand bytes (and L2 requests, of which such rows need twice as many) per flop, measured +4.5 to +6.7 % at
  // 12288 x 6144, 6144 x 12288, 12288 x 12288, 3072 x 3072 and 6144 x 3072 (x 1000), +0.5 to +1.7 % at 6144 x 6144,
  // 3072 x 12288 and 12288 x 3072, but -2.6 % with four tile rows (2048 x 12288); with an fp32 C or rows on the grid
  // (K = 1024) its exposed epilogue loses.
  if (best_g == 2 && best_n == 256 && best_p == 1 && best_r == 1 && unaligned_rows && c.c_bytes == 2 && c.batch <= 1 &&
      c.K * (c.ab_bytes / 2) >= 768 && c.K * (c.ab_bytes / 2) <= 1536 && c.M >= 3072 && c.N >= 3072 && max_pairs >= 1 &&
      o.mrep == 0 && o.cta_group == 0 && o.tile_n == 0 && o.share == 0 && o.ksub != 2 && !o.reduce_add && o.grid_limit == 0)
    best_r = 2;
  // Where the choice fell on plain pairs of 256 x 256 tiles and the operand rows are not 128-byte aligned,
  // the same tiles in shared-operand clusters are the faster form (see kShareGainUnalignedRows), unless the
  // slots of two tiles quantise worse than the single tiles did.
  // (The library's own tile choices only: a caller who names a tile shape gets plain pairs unless the
  // clusters are asked for as well.)
  // The same where the tail of the plain pairs would be shared out in ranges that ignore tile boundaries:
  // the two pairs of a cluster work on neighbouring tiles at the same k-blocks, which gives back part of the
  // operand sharing in L2 that such ranges lose (3072 x 1000 x 12288 +7.8 %, 12288 x 1000 x 6144 +5.2 %,
  // 6144 x 2048 x 6144 +3.2 %, 6144 x 512 x 12288 +2 %).
  bool ranges = false;
  if (best_g == 2 && best_n == 256 && best_p == 1 && best_r == 1 && max_pairs >= 1) {
    int64_t w_pairs = max_pairs;
    if (o.grid_limit && o.grid_limit / 2 < w_pairs) w_pairs = o.grid_limit / 2;
    const int64_t tiles_pairs = ((c.M + 255) / 256) * ((c.N + 255) / 256) * c.batch;
    if (w_pairs >= 1) {
      const int64_t tail = tiles_pairs % w_pairs;
      const int tw = tail_workers_for(tiles_pairs, w_pairs, c.K * (c.ab_bytes / 2), default_ksub(2, 256), o, 1);
      ranges = tw > 0 && tail > 0 && tw % tail != 0;
    }
  }
  if (best_g == 2 && best_n == 256 && best_p == 1 && best_r == 1 && o.share == 0 && (unaligned_rows || ranges) && max_quads >= 1 &&
      o.cta_group == 0 && o.tile_n == 0 && o.mrep == 0 && !o.reduce_add && (o.grid_limit & 3) == 0) {
    int w_eff = max_quads;
    if (o.grid_limit && o.grid_limit / 4 < w_eff) w_eff = o.grid_limit / 4;
    if (w_eff >= 1) {
      const double t = estimate_clocks(c.M, c.N, c.K * (c.ab_bytes / 2), c.batch, 2, 256, w_eff, o, 2, 1,
                                       c.a_mn_major || c.b_mn_major, true);
      if (t <= best * (ranges ? 1.03 : 1.0)) best_p = 2;
    }
  }
  // Problems of less than one wave: the one-tile-per-CTA kernel (lean_kernel.cuh), 128 x 64 tiles while they
  // fit the SMs at one per SM, else 128 x 128.
  bool lean = false;
  int lean_split = 1;   // CTAs (a cluster) that share a lean tile's K loop: 1, 2 or 4
  if (o.lean == 2 && o.cta_group == 2 && c.batch <= 1 && max_pairs >= 1) {   // on request: a CTA pair per 256 x N tile
    lean = true;
    best_g = 2; best_n = o.tile_n ? o.tile_n : 256; best_p = 1; best_r = 1;
  } else if (o.lean != 1 && c.batch <= 1 && !o.reduce_add && o.share < 2 && o.mrep != 2 && o.cta_group != 2 && o.tile_n != 256 &&
      o.grid_limit == 0 && (o.split < 2 || o.split == 2 || o.split == 4)) {
    const int ksub = o.ksub ? o.ksub : 2;
    const int64_t nkb_all = (c.K * (c.ab_bytes / 2) + kBlockK * ksub - 1) / (kBlockK * ksub);
    int bn = 64, split = 1;
    if (o.lean == 2) {   // on request: 128 x 64 tiles while a CTA per tile fits the SMs, else 128 x 128; K cut as asked
      const int64_t t64 = ((c.M + 127) / 128) * ((c.N + 63) / 64);
      bn = o.tile_n ? o.tile_n : (t64 <= sm_count ? 64 : 128);
      split = o.split >= 2 ? o.split : 1;
      lean = true;
    } else if (o.tile_n == 0 && o.cta_group == 0 && o.ksub == 0 && o.stages == 0 && o.epi_bufs == 0 && o.band == 0 &&
               o.along_m == 0 && o.split < 2) {
      // (the library's own choice only where the caller names no parameter of the persistent kernel)
      lean = lean_is_faster(c, o, sm_count, &bn, &split);
    }
    if (lean) {
      best_g = 1; best_n = bn; best_p = 1; best_r = 1;
      lean_split = split;
      while (lean_split > 1 && lean_split > nkb_all) lean_split /= 2;   // every CTA of a cluster gets a k-block
      const int64_t lean_tiles = ((c.M + 127) / 128) * ((c.N + bn - 1) / bn);
      while (lean_split > 1 && lean_tiles * lean_split >= (1LL << 31)) lean_split /= 2;   // the grid is indexed with 32 bits
    }
  }
  TileConfig cfg;
  cfg.lean = lean ? lean_split : 0;
  cfg.cta_group = best_g;
  cfg.tile_n = best_n;
  cfg.pairs = best_p;
  cfg.mrep = best_r;
  cfg.ksub = best_r == 2 ? 1 : (o.ksub ? o.ksub : default_ksub(best_g, best_n));
  cfg.tiles_m = (int)((c.M + 128 * best_g * best_r - 1) / (128 * best_g * best_r));
  cfg.tiles_n = (int)((c.N + best_n * best_p - 1) / (best_n * best_p));
  int64_t workers = best_p == 2 ? max_quads : (best_g == 2 ? max_pairs : sm_count);
  if (o.grid_limit && o.grid_limit / (best_g * best_p) < workers) workers = o.grid_limit / (best_g * best_p);
  if (workers < 1) workers = 1;
  const int64_t tiles = (int64_t)cfg.tiles_m * cfg.tiles_n * c.batch;
  if (lean) workers = tiles < 1 ? 1 : tiles;   // a cluster per tile, all at once
  // Two staging buffers per epilogue warp let a warp fill one while the TMA store still
  // reads the other; they cost 32 KB of ring.  Short K: the epilogue bounds a tile, so staging
  // depth matters more than ring depth.  Otherwise the ring takes the space: the time between a
  // stage's release and its reuse has to cover a commit, the producer's wake-up and an L2 or DRAM
  // round trip (measured: 6 stages instead of 5 give +1.3 to +4.6 % for K >= 2048).
  // A 16-bit C halves the epilogue's stores, and one buffer with the deeper ring is then at least level at
  // every K (bf16 C, 6 stages + 1 buffer against 5 + 2: +3 to +5 % at K = 1000 .. 1024, +1 % at 512 and 1536,
  // -0.2 % at 12288 x 12288 x 512).
  const int64_t k16 = c.K * (c.ab_bytes / 2);
  // (except at K <= 512 with fewer than three tiles per worker, where the second buffer measured +1 to +3 %)
  const bool want_two = (c.c_bytes == 4 ? k16 <= 1024 : (k16 <= 512 && tiles < 3 * workers)) &&
                        max_stages(best_g, best_n, cfg.ksub, 2, best_r) >= 3;
  cfg.epi_bufs = o.epi_bufs ? o.epi_bufs : (want_two ? 2 : 1);
  cfg.stages = max_stages(best_g, best_n, cfg.ksub, cfg.epi_bufs, best_r);
  if (o.stages && o.stages < cfg.stages) cfg.stages = o.stages < 2 ? 2 : o.stages;
  cfg.stages_direct = (o.epi_bufs || o.reduce_add) ? 0 : max_stages(best_g, best_n, cfg.ksub, 0, best_r);
  if (o.stages && o.stages < cfg.stages_direct) cfg.stages_direct = o.stages < 2 ? 2 : o.stages;
  if (lean) {  // a ring no deeper than a CTA's K loop: with every k-block resident no stage is ever waited for
    const int64_t nkb_all = (k16 + kBlockK * cfg.ksub - 1) / (kBlockK * cfg.ksub);
    const int64_t nkb = (nkb_all + lean_split - 1) / lean_split;
    cfg.stages = best_g == 2 ? lean_pair_max_stages(best_n, cfg.ksub) : lean_max_stages(best_n, cfg.ksub, c.c_bytes, lean_split);
    if (nkb < cfg.stages) cfg.stages = nkb < 1 ? 1 : (int)nkb;
    if (o.stages && o.stages < cfg.stages) cfg.stages = o.stages;
    // (a cluster's CTAs stage their partial sums, 4 quadrants x 128 bytes x tile_n, in the ring once their MMAs are done)
    while (lean_split > 1 && cfg.stages * stage_bytes(1, best_n, cfg.ksub) < 16 * best_n * 32) ++cfg.stages;
    cfg.stages_direct = 0;
    cfg.epi_bufs = 1;
  }
  // Wave quantisation: the k-blocks of the tiles that do not fill a whole wave are shared out evenly among
  // the workers, so that the last wave takes tail / tail_workers of a tile's time (split-K applied to the
  // tail only; for a problem smaller than one wave that is split-K with slices of equal length).
  {
    const int64_t full_waves = tiles / workers;
    cfg.full_tiles = full_waves * workers;
    cfg.tail_tiles = (int)(tiles - cfg.full_tiles);
    const int64_t k_scaled = c.K * (c.ab_bytes / 2);  // in 16-bit-element units: 64 per sub-block
    cfg.tail_workers = tail_workers_for(tiles, workers, k_scaled, cfg.ksub, o, best_r);
    cfg.slots = 0;
    cfg.snap = 0;
    cfg.owner_extra = 0;
    cfg.split = 1;
    if (cfg.tail_workers > 0) {   // the exact slot count comes from the table of ranges
      const int32_t nkb = (int32_t)((k_scaled + kBlockK * cfg.ksub - 1) / (kBlockK * cfg.ksub));
      TailItem* table = new TailItem[4 * (size_t)workers];
      cfg.snap = o.split >= 2 ? 0 : tail_snap(cfg.ksub);   // a requested slice count is taken literally
      // In a problem of less than one wave all slices run side by side: publishing a 128 x N fp32 partial
      // takes a contributor about as long as 8 k-blocks of 64 (128*N*4 bytes at ~30 B/clk against 2*N
      // clocks of MMA per k-block), so there the owner computes that much longer.
      if (cfg.full_tiles == 0 && cfg.tail_workers % cfg.tail_tiles == 0) {
        const int64_t f = cfg.tail_workers / cfg.tail_tiles;
        int64_t extra = 8 / cfg.ksub;
        const int64_t room = nkb / f - 1;   // every other slice keeps at least one k-block
        if (extra > room / 2) extra = room / 2;
        cfg.owner_extra = (int)(extra < 0 ? 0 : extra);
      }
      cfg.slots = build_tail_table(cfg.tail_tiles, nkb, cfg.tail_workers, (int32_t)workers, table, cfg.snap, cfg.owner_extra);
      delete[] table;
      cfg.split = cfg.slots + 1;
      if (cfg.slots == 0) cfg.tail_workers = 0;
    }
    cfg.workspace_bytes = 0;  // filled in by split_workspace_bytes() once the output type is known
  }
  // One whole tile per worker and nothing after it: the drain is exposed, and with a single staging buffer a
  // warp waits about 1000 clocks per chunk for the previous store to have read it.  fp32 C, 5 stages + 2 buffers
  // against 6 + 1: 2048^3 -3.1 %, 2048 x 2048 x 3072 -2.7 %, 1000 x 3072 x 3072 -3.3 %, 2048 x 2048 x 6144 -0.8 % (time);
  // with a 16-bit C -1 %, not taken.
  // (256-column tiles, where it was measured: a ring of 32 KB stages goes from 6 to 5; narrower tiles would go from 4 to 3)
  if (!lean && !o.epi_bufs && c.c_bytes == 4 && best_r == 1 && best_n == 256 && cfg.full_tiles == 0 && cfg.tail_workers == 0 && cfg.epi_bufs == 1 &&
      max_stages(best_g, best_n, cfg.ksub, 2, best_r) >= 3) {
    cfg.epi_bufs = 2;
    cfg.stages = max_stages(best_g, best_n, cfg.ksub, 2, best_r);
    if (o.stages && o.stages < cfg.stages) cfg.stages = o.stages < 2 ? 2 : o.stages;
  }
  if (tiles < workers) {  // less than one wave: launch only the CTA groups that get a work item
    workers = cfg.tail_workers > 0 ? cfg.tail_workers : tiles;
    if (workers < 1) workers = 1;
  }
  cfg.workers = (int)workers;
  cfg.along_m = o.along_m;
  // Ranges of the tail's k-blocks that ignore tile boundaries put consecutive tiles on consecutive workers,
  // a fraction of a tile out of step: the operand panel that neighbouring tiles share stays in L2 only if
  // it is the small one, so the raster walks the shorter side of the tile grid first (6144 x 512 x 12288:
  // +9 % with bands along M, 512 x 6144 x 12288: -9 %; with whole tiles the direction measured +-0.5 %).
  if (cfg.tail_workers > 0 && cfg.tail_workers % cfg.tail_tiles != 0 && cfg.tiles_m > cfg.tiles_n) cfg.along_m = 1;
  // A grid of few tile rows and many tile columns behind a long K loop: bands that span all the rows and walk N
  // (the mirror image of what a tall grid gets by default) measured +2.0 % at 1024 x 16384 x 4096, +2.3 % at
  // 2048 x 6144 x 6144, +1.6 % at 1000 x 12288 x 12288, +0.5 to +0.8 % at 2048 x 12288 x 2048 and 512 x 12288 x 6144;
  // with more rows or a short K the direction measured +-0.5 %.
  if (!lean && best_p == 1 && cfg.tiles_m <= 8 && cfg.tiles_n >= 3 * cfg.tiles_m && k16 >= 2048) cfg.along_m = 1;
  // Tiles that run together should cover a square patch of C: band width G along
  // the banded dimension minimises (W/G)*extent_other + G*extent_banded.
  const double tile_m = 128.0 * best_g * best_r, tile_n = (double)best_n * best_p;
  const double ratio = cfg.along_m ? tile_n / tile_m : tile_m / tile_n;
  int band = o.band ? o.band : (int)floor(sqrt((double)workers * ratio) + 0.5);
  const int major = cfg.along_m ? cfg.tiles_m : cfg.tiles_n;
  if (band > major) band = major;
  if (band > 15) band = 15;
  if (band < 1) band = 1;
  cfg.band = band;
  return cfg;
}

// Bytes of fp32 partials: per tail tile and slice beyond the first, every epilogue warp of every
// CTA of the group stores its chunks as 4 KB units (32 rows x 32 fp32 columns).
inline int64_t split_workspace_bytes(const TileConfig& cfg, int c_dtype) {
  if (cfg.tail_workers <= 0) return 0;
  const int cw = c_dtype == EXO_GEMM_FP32 ? 32 : 64;        // columns per epilogue chunk
  const int nchunk = cfg.tile_n / cw;
  const int units_per_warp = ((nchunk + 1) / 2) * (cw / 32);
  return (int64_t)cfg.tail_tiles * cfg.slots * cfg.cta_group * cfg.pairs * cfg.mrep * kEpiWarps * units_per_warp * 4096;
}

inline int smem_bytes_for(int cta_group, int bn, int ksub, int stages, int epi_bufs, int mrep = 1) {
  return 1024 + stages * stage_bytes(cta_group, bn, ksub, mrep) + kEpiWarps * epi_bufs * kEpiBufBytes + kBarrierBytes;
}

// tcgen05 instruction descriptor for kind::f16 with fp32 accumulation.
inline uint32_t make_idesc(int ab_dtype, int a_mn_major, int b_mn_major, int umma_m, int umma_n) {
  // kind::f16: 0 = fp16, 1 = bf16; kind::tf32: 2 = tf32
  const uint32_t fmt = ab_dtype == EXO_GEMM_BF16 ? 1u : (ab_dtype == EXO_GEMM_FP32 ? 2u : 0u);
  uint32_t d = 0;
  d |= 1u << 4;                        // D format: fp32
  d |= fmt << 7;                       // A format
  d |= fmt << 10;                      // B format
  d |= (uint32_t)(a_mn_major & 1) << 15;
  d |= (uint32_t)(b_mn_major & 1) << 16;
  d |= (uint32_t)(umma_n >> 3) << 17;
  d |= (uint32_t)(umma_m >> 4) << 24;
  return d;
}

// How an operand tile sits in shared memory (128-byte swizzle, 8-row atoms of 1 KB).
inline OperandStaging make_staging(int mn_major, int rows, int ksub, int ab_bytes) {
  OperandStaging s;
  s.mn_major = (uint32_t)mn_major;
  const uint32_t sbo = 1024u >> 4;       // between 8-row groups of a swizzle atom column
  const uint32_t version = 1u << 14;     // descriptor bits 46..47 = 1 on sm_100
  const uint32_t swizzle128 = 2u << 29;  // descriptor bits 61..63
  s.desc_hi = sbo | version | swizzle128;
  if (!mn_major) {
    s.lbo_enc = 1;                                   // unused for swizzled K-major tiles
    s.k_step_enc = (kUmmaK * 2) >> 4;                // 32 bytes along the 128-byte row
    s.k_sub_enc = ((uint32_t)rows * 128u) >> 4;      // next sub-block: next box of `rows` rows
  } else {
    const uint32_t sub_k = (uint32_t)sub_block_k(ab_bytes);   // k-rows per sub-block: 64 or 32
    const uint32_t umma_k = sub_k / 4;                        // k-rows per MMA: 16 or 8
    if (ab_bytes == 4) {
      // An M/N-contiguous 32-bit operand takes the 128-byte swizzle with 32-byte atomicity (the pattern
      // repeats every 4 rows of 128 bytes, not every 8): layout type 1 and a 512-byte stride between
      // groups of 4 k-rows; the TMA maps of such operands use the matching swizzle mode.
      s.desc_hi = (512u >> 4) | version | (1u << 29);
    }
    // one TMA box per group of 128 bytes of M/N elements: sub_k*ksub k-rows of 128 bytes; the kernel
    // issues rows / 64 of them per stage (16-bit operands; fp32 operands are K-contiguous only)
    const uint32_t box_bytes = (uint32_t)ksub * sub_k * 128u;
    s.lbo_enc = box_bytes >> 4;                      // next group of M/N elements: next box
    s.k_step_enc = (umma_k * 128u) >> 4;             // the k-rows of one MMA
    s.k_sub_enc = (sub_k * 128u) >> 4;               // k-rows continue inside the same box
  }
  return s;
}

}  // namespace exo
