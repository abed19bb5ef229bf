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
// waves can be filled (`full_tiles` = the largest multiple of the worker count
// not above the tile count).  The `tail_tiles` tiles left over would occupy only
// part of a last wave, so each of them is cut along K into `split` slices and
// the tail_tiles * split <= num_workers units are dealt one per worker: the
// last wave then takes about 1/split of a tile's time.  (The paper's Section 6
// kernels use split-K for the same wave-quantisation problem; here the split is
// applied only where it pays, and the reduction order is fixed.)  split == 1
// degenerates to plain round-robin.
struct WorkPlan {
  int64_t full_tiles;   // tiles [0, full_tiles) are whole-K work items
  int32_t tail_tiles;   // tiles [full_tiles, full_tiles + tail_tiles) are cut into slices
  int32_t split;        // slices per tail tile, >= 1
  int32_t owner_extra;  // k-blocks slice 0 takes beyond an even share: the other slices finish
                        // earlier by about the time it takes them to publish their partial sums
};

struct WorkItem {
  int64_t tile;         // linear tile index (to be decoded by raster_decode)
  int32_t tail_index;   // index among the tail tiles, or -1 for a whole-K item
  int32_t slice;        // 0 .. slices - 1; slice 0 owns the output tile
  int32_t slices;
  int32_t kb_begin, kb_end;  // k-blocks [kb_begin, kb_end) of num_k_blocks
};

// The i-th work item of `worker`; returns false when the worker has no i-th item.
// A worker whose unit of a tail tile is a contributing slice (slice > 0) computes that unit FIRST and
// its whole tiles afterwards: its partial sums then reach memory a whole tile's time before the owning
// slice (slice 0, computed LAST by its worker) asks for them, and neither side ever waits.
// The owners are workers 0 .. tail_tiles-1 and the contributors the workers after them: a worker that
// starts with a slice stays out of step with the others for the whole launch, and tiles that run in step
// share their operand panels in L2, so each group is kept contiguous in the tile order.
EXO_HD bool work_item(const WorkPlan& w, int64_t worker, int64_t num_workers, int64_t i, int32_t num_k_blocks,
                      WorkItem* out) {
  const bool has_unit = worker < (int64_t)w.tail_tiles * w.split;
  const bool early = has_unit && worker >= w.tail_tiles;  // a contributing slice (split > 1 follows)
  if (!(early && i == 0)) {
    const int64_t t = worker + (early ? i - 1 : i) * num_workers;
    if (t < w.full_tiles) {
      out->tile = t;
      out->tail_index = -1;
      out->slice = 0;
      out->slices = 1;
      out->kb_begin = 0;
      out->kb_end = num_k_blocks;
      return true;
    }
    if (early || !has_unit) return false;
    if (t - w.full_tiles != worker) return false;           // only the wave right after the full ones
  }
  const int32_t sl = (int32_t)((uint32_t)worker / (uint32_t)w.tail_tiles);
  const int32_t ti = (int32_t)((uint32_t)worker - (uint32_t)sl * (uint32_t)w.tail_tiles);
  out->tile = w.full_tiles + ti;
  out->tail_index = w.split > 1 ? ti : -1;
  out->slice = sl;
  out->slices = w.split;
  // slice 0: an even share plus owner_extra; slices 1.. share the rest evenly, in K order
  int32_t own = (num_k_blocks + w.split - 1) / w.split + (w.split > 1 ? w.owner_extra : 0);
  if (own > num_k_blocks - (w.split - 1)) own = num_k_blocks - (w.split - 1);
  if (own < 1) own = 1;
  if (w.split == 1) own = num_k_blocks;
  if (sl == 0) {
    out->kb_begin = 0;
    out->kb_end = own;
  } else {
    const uint32_t rest = (uint32_t)(num_k_blocks - own);   // rest * slice < 2^31: both are small
    out->kb_begin = own + (int32_t)((rest * (uint32_t)(sl - 1)) / (uint32_t)(w.split - 1));
    out->kb_end = own + (int32_t)((rest * (uint32_t)sl) / (uint32_t)(w.split - 1));
  }
  return true;
}

}  // namespace exo
