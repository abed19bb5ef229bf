// Persistent tile scheduler: static round-robin over a band-swizzled raster.
//
// The paper's generated kernels launch just enough clusters to fill the device
// and hand them tasks round-robin in lexicographic order (Section 4.2,
// "persistent kernel" / task generator), and name a swizzled order as future
// work.  Here worker w of W visits linear indices w, w + W, w + 2W, ...; a linear
// index is mapped to a tile through bands: with bands along N (along_m == 0) the
// tile grid is cut into bands of `band` tile columns, and inside a band the
// index walks the band's columns first, then the next tile row.  The tiles that
// run at the same time then cover a roughly square patch of C, so the rows of A
// and columns of B they stream are shared through L2.  along_m == 1 is the
// transposed raster.
//
// Plain functions, usable on host and device.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define EXO_HD __host__ __device__ __forceinline__
#else
#define EXO_HD inline
#endif

namespace exo {

struct TileCoord {
  int32_t m, n;
};

// Division of a 31-bit numerator by a divisor fixed per launch, as a multiply and a shift (the
// round-up method: m = ceil(2^(31+l) / d) with l = ceil(log2 d) gives floor(n / d) exactly for every
// n < 2^31).  A hardware division costs the scheduling warps about a hundred clocks at every tile.
struct FastDiv {
  uint32_t mul, shift;   // shift == 32: the divisor is 1
};

inline FastDiv make_fast_div(uint32_t d) {
  FastDiv f;
  if (d <= 1) { f.mul = 0; f.shift = 32; return f; }
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;                                   // ceil(log2 d) >= 1
  f.mul = (uint32_t)((((uint64_t)1 << (31 + l)) + d - 1) / d);   // <= 2^32 - 1 for d >= 2
  f.shift = l - 1;
  return f;
}

EXO_HD uint32_t fast_div(uint32_t n, const FastDiv& f) {
#if defined(__CUDA_ARCH__)
  return f.shift == 32u ? n : (__umulhi(n, f.mul) >> f.shift);
#else
  return f.shift == 32u ? n : (uint32_t)(((uint64_t)n * f.mul) >> 32) >> f.shift;
#endif
}

struct Raster {
  int32_t tiles_m, tiles_n;
  int32_t band;      // >= 1
  int32_t along_m;   // 0: bands are groups of tile columns; 1: groups of tile rows
  FastDiv by_per_band, by_band, by_last;   // divisions by band * minor, by band and by the last band's width
};

// The raster of a tiles_m x tiles_n grid with its division constants (host side).
inline Raster make_raster(int32_t tiles_m, int32_t tiles_n, int32_t band, int32_t along_m) {
  Raster r;
  r.tiles_m = tiles_m;
  r.tiles_n = tiles_n;
  r.band = band < 1 ? 1 : band;
  r.along_m = along_m ? 1 : 0;
  const uint32_t major = (uint32_t)(r.along_m ? tiles_m : tiles_n);
  const uint32_t minor = (uint32_t)(r.along_m ? tiles_n : tiles_m);
  const uint32_t last = major % (uint32_t)r.band;
  r.by_per_band = make_fast_div((uint32_t)r.band * (minor ? minor : 1u));
  r.by_band = make_fast_div((uint32_t)r.band);
  r.by_last = make_fast_div(last ? last : (uint32_t)r.band);
  return r;
}

EXO_HD int64_t raster_total(const Raster& r) { return (int64_t)r.tiles_m * r.tiles_n; }

// linear index -> tile coordinate.  Tile counts stay below 2^31 (checked by the host plan), so
// the arithmetic is 32-bit, and the divisions are multiplications by constants the host prepared:
// they sit on the critical path of every tile.
EXO_HD TileCoord raster_decode(const Raster& r, int64_t t64) {
  const uint32_t t = (uint32_t)t64;
  // "major" = the banded dimension, "minor" = the other one
  const uint32_t major = (uint32_t)(r.along_m ? r.tiles_m : r.tiles_n);
  const uint32_t minor = (uint32_t)(r.along_m ? r.tiles_n : r.tiles_m);
  const uint32_t per_band = (uint32_t)r.band * minor;
  const uint32_t b = fast_div(t, r.by_per_band);
  const uint32_t in_band = t - b * per_band;
  const uint32_t first = b * (uint32_t)r.band;
  const bool narrow = (major - first) < (uint32_t)r.band;         // the last band may be narrower
  const uint32_t width = narrow ? (major - first) : (uint32_t)r.band;
  const uint32_t i_minor = fast_div(in_band, narrow ? r.by_last : r.by_band);
  const uint32_t i_major = first + (in_band - i_minor * width);
  TileCoord c;
  c.m = (int32_t)(r.along_m ? i_major : i_minor);
  c.n = (int32_t)(r.along_m ? i_minor : i_major);
  return c;
}

// ---------------------------------------------------------------------------
// Work list of one worker.  Tiles are dealt round-robin for as long as whole
// waves can be filled (`waves` waves of `num_workers` tiles).  The `tail_tiles`
// tiles left over would occupy only part of a last wave.  Their k-blocks,
// tail_tiles * num_k_blocks in tile-major order, are instead cut into
// `tail_workers` equal consecutive ranges, one per worker: a range covers the
// end of one tile and the beginning of the next, so a tile is computed by two
// or more workers whatever the ratio of tiles to workers is, and the last wave
// takes tail_tiles / tail_workers of a tile's time.  (The paper's Section 6
// kernels use split-K against the same wave-quantisation problem; this is
// split-K applied to the tail only, with slices that need not end at tile
// boundaries, and with a fixed reduction order.)  The part of a tile that
// starts at k-block 0 is the owning slice: its worker adds the other parts'
// partial sums, in K order, and writes the tile.  tail_workers == 0: the tail
// tiles are whole-K items like the others.
//
// The ranges are laid out by the host into a table of four 16-byte entries per
// worker -- {items that come first, items in all, -, -} and up to three items
// -- because finding them takes 64-bit divisions that no role should repeat at
// every tile.
struct TailItem {
  int32_t tail_index;  // which tail tile (the tile is full_tiles + tail_index)
  int32_t kb_begin, kb_end;
  int32_t slice_info;  // slice | slices << 16: slice 0 owns the tile, slices - 1 others contribute to it
};

struct WorkPlan {
  int64_t full_tiles;    // tiles [0, full_tiles) are whole-K work items: waves * num_workers
  int32_t waves;
  int32_t tail_tiles;    // tiles [full_tiles, full_tiles + tail_tiles)
  int32_t tail_workers;  // workers that share the tail tiles' k-blocks (0: the tail is not cut)
  int32_t slots;         // partial-sum slots per tail tile in the workspace: the most contributors any tile has
  int32_t owner_extra;   // whole slices: k-blocks the owning slice takes beyond an even share
  const TailItem* table; // ranges: device (or host, for the host-side enumeration) table, 4 entries per worker;
                         // NULL: tail_workers is a multiple of tail_tiles and every tile is cut into whole slices
};

struct WorkItem {
  int64_t tile;         // linear tile index (to be decoded by raster_decode)
  int32_t tail_index;   // index among the tail tiles, or -1 for a whole-K item
  int32_t slice;        // 0 .. slices - 1 in K order; slice 0 owns the output tile
  int32_t slices;       // parts the tile is cut into (1: a whole-K item)
  int32_t kb_begin, kb_end;  // k-blocks [kb_begin, kb_end) of num_k_blocks
  int32_t after_whole;  // 1: the item before this one (of the same worker) is a whole tile
};

// Fills the table (4 * num_workers entries) and returns the number of slots per tail tile.
// Needs tail_tiles <= tail_workers <= num_workers and tail_workers <= tail_tiles * num_k_blocks.
// A range boundary that falls within `snap` k-blocks of a tile boundary is moved onto it: a part of a
// few k-blocks saves less main-loop time than the exchange of its partial sums costs.
//
// Where the sharing workers are a multiple f of the tail tiles, every tile is cut into f slices at the
// same k-blocks instead, slice s of tile t goes to worker s * tail_tiles + t, and the owning slice takes
// `owner_extra` k-blocks more than an even share (for problems of less than one wave, where all slices
// run side by side and the others need time to publish their sums).  The owners are then workers
// 0 .. tail_tiles - 1 and the contributors the workers after them: a worker that starts with a slice stays
// out of step with the others for the whole launch, and tiles that run in step share their operand panels
// in L2, so each group is kept contiguous in the tile order (measured: +0.5 % against -1 to -2.8 % with
// owners and contributors interleaved).
inline int32_t build_tail_table(int32_t tail_tiles, int32_t num_k_blocks, int32_t tail_workers, int32_t num_workers,
                                TailItem* table, int32_t snap = 0, int32_t owner_extra = 0) {
  if (tail_workers % tail_tiles == 0) {
    const int32_t f = tail_workers / tail_tiles;
    int32_t own = (num_k_blocks + f - 1) / f + (f > 1 ? owner_extra : 0);
    if (own > num_k_blocks - (f - 1)) own = num_k_blocks - (f - 1);
    if (own < 1) own = 1;
    if (f == 1) own = num_k_blocks;
    for (int32_t w = 0; w < num_workers; ++w) {
      TailItem* e = table + 4 * w;
      for (int k = 0; k < 4; ++k) e[k] = TailItem{0, 0, 0, 0};
      if (w >= tail_workers) continue;
      const int32_t sl = w / tail_tiles;
      TailItem it;
      it.tail_index = w - sl * tail_tiles;
      it.slice_info = sl | (f << 16);
      if (sl == 0) {
        it.kb_begin = 0;
        it.kb_end = own;
      } else {   // slices 1.. share the rest evenly, in K order
        const int64_t rest = num_k_blocks - own;
        it.kb_begin = own + (int32_t)(rest * (sl - 1) / (f - 1));
        it.kb_end = own + (int32_t)(rest * sl / (f - 1));
      }
      e[1] = it;
      e[0].tail_index = sl > 0 ? 1 : 0;   // contributing slices come first
      e[0].kb_begin = 1;
    }
    return f - 1;
  }
  const int64_t units = (int64_t)tail_tiles * num_k_blocks;
  if (snap > num_k_blocks / 8) snap = num_k_blocks / 8;
  if (snap > units / tail_workers / 4) snap = (int32_t)(units / tail_workers / 4);   // never a whole range
  int64_t* bound = new int64_t[(size_t)tail_workers + 1];
  for (int32_t j = 0; j <= tail_workers; ++j) {
    int64_t b = (int64_t)j * units / tail_workers;
    const int64_t r = b % num_k_blocks;
    if (r != 0 && r <= snap) b -= r;
    else if (r != 0 && num_k_blocks - r <= snap) b += num_k_blocks - r;
    bound[j] = b;
  }
  // the worker whose range holds unit u (ranges may be empty after snapping: the last one that starts at or before u)
  auto holder = [&](int64_t u) {
    int32_t j = (int32_t)((u * tail_workers) / units);
    if (j > tail_workers - 1) j = tail_workers - 1;
    while (j + 1 < tail_workers && bound[j + 1] <= u) ++j;
    while (j > 0 && bound[j] > u) --j;
    return j;
  };
  int32_t slots = 0;
  for (int32_t w = 0; w < num_workers; ++w) {
    TailItem* e = table + 4 * w;
    for (int k = 0; k < 4; ++k) e[k] = TailItem{0, 0, 0, 0};
    if (w >= tail_workers) continue;
    const int64_t b0 = bound[w], b1 = bound[w + 1];
    int32_t n = 0, lead = 0;
    TailItem late[2];
    int32_t n_late = 0;
    for (int64_t a = b0 / num_k_blocks; a * num_k_blocks < b1 && n + n_late < 3; ++a) {
      const int64_t lo = a * num_k_blocks, hi = lo + num_k_blocks;
      TailItem it;
      it.tail_index = (int32_t)a;
      it.kb_begin = (int32_t)((b0 > lo ? b0 : lo) - lo);
      it.kb_end = (int32_t)((b1 < hi ? b1 : hi) - lo);
      // the tile's parts are the non-empty ranges from the one that holds its first k-block (the owner)
      // to the one that holds its last; this part's number among them is its place in K order
      const int32_t first = holder(lo), last = holder(hi - 1);
      int32_t slice = 0, parts = 0;
      for (int32_t j = first; j <= last; ++j) {
        if (bound[j + 1] <= bound[j]) continue;
        if (j < w) ++slice;
        ++parts;
      }
      if (parts - 1 > slots) slots = parts - 1;
      it.slice_info = slice | (parts << 16);
      if (it.kb_begin > 0) { e[1 + n++] = it; ++lead; }   // a contributing part: computed first
      else if (n_late < 2) late[n_late++] = it;            // whole tiles and owning parts: computed last
    }
    for (int32_t k = 0; k < n_late; ++k) e[1 + n++] = late[k];
    e[0].tail_index = lead;
    e[0].kb_begin = n;
  }
  delete[] bound;
  return slots;
}

// The i-th work item of `worker`; returns false when the worker has no i-th item.
// A worker's contributing part of a tail tile (it does not start at k-block 0) comes FIRST and its whole
// tiles afterwards: the partial sums then reach memory a whole tile's time before the owning part
// (computed LAST by its worker) asks for them, and neither side ever waits.
EXO_HD bool work_item(const WorkPlan& w, int64_t worker, int64_t num_workers, int64_t i, int32_t num_k_blocks,
                      WorkItem* out) {
  int32_t lead = 0, n_items = 0;
  const TailItem* e = nullptr;
  // whole slices: every sharing worker has exactly one part, found by arithmetic (the table is for ranges
  // only: its two dependent loads would sit in front of the first copy of every worker of a small problem)
  const bool whole_slices = w.tail_workers > 0 && w.table == nullptr;
  if (whole_slices) {
    n_items = worker < w.tail_workers ? 1 : 0;
    lead = n_items && worker >= w.tail_tiles ? 1 : 0;   // a contributing slice
  } else if (w.tail_workers > 0) {
    e = w.table + 4 * worker;
    lead = e[0].tail_index;
    n_items = e[0].kb_begin;
  }
  int64_t k;   // index into this worker's tail items, if the i-th item is one
  if (i < lead) {
    k = i;
  } else {
    const int64_t j = i - lead;
    const int64_t t = worker + j * num_workers;
    if (j < w.waves || (w.tail_workers == 0 && t < w.full_tiles + w.tail_tiles)) {
      out->tile = t;
      out->tail_index = -1;
      out->slice = 0;
      out->slices = 1;
      out->kb_begin = 0;
      out->kb_end = num_k_blocks;
      out->after_whole = j >= 1;
      return true;
    }
    k = lead + (j - w.waves);
    if (w.tail_workers == 0 || k >= n_items) return false;
  }
  out->after_whole = i > lead;   // (items that come first have no whole tile before them)
  if (whole_slices) {
    const int32_t f = w.slots + 1;
    const int32_t sl = (int32_t)((uint32_t)worker / (uint32_t)w.tail_tiles);
    const int32_t ti = (int32_t)((uint32_t)worker - (uint32_t)sl * (uint32_t)w.tail_tiles);
    out->tile = w.full_tiles + ti;
    out->tail_index = ti;
    out->slice = sl;
    out->slices = f;
    // slice 0: an even share plus owner_extra; slices 1.. share the rest evenly, in K order
    int32_t own = (num_k_blocks + f - 1) / f + w.owner_extra;
    if (own > num_k_blocks - (f - 1)) own = num_k_blocks - (f - 1);
    if (own < 1) own = 1;
    if (sl == 0) {
      out->kb_begin = 0;
      out->kb_end = own;
    } else {
      const uint32_t rest = (uint32_t)(num_k_blocks - own);   // rest * slice < 2^31: both are small
      out->kb_begin = own + (int32_t)((rest * (uint32_t)(sl - 1)) / (uint32_t)(f - 1));
      out->kb_end = own + (int32_t)((rest * (uint32_t)sl) / (uint32_t)(f - 1));
    }
    return true;
  }
  const TailItem it = e[1 + k];
  out->tile = w.full_tiles + it.tail_index;
  out->slice = it.slice_info & 0xFFFF;
  out->slices = it.slice_info >> 16;
  out->tail_index = out->slices > 1 ? it.tail_index : -1;
  out->kb_begin = it.kb_begin;
  out->kb_end = it.kb_end;
  return true;
}

}  // namespace exo
