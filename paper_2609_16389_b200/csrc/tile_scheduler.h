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

struct Raster {
  int32_t tiles_m, tiles_n;
  int32_t band;      // >= 1
  int32_t along_m;   // 0: bands are groups of tile columns; 1: groups of tile rows
};

EXO_HD int64_t raster_total(const Raster& r) { return (int64_t)r.tiles_m * r.tiles_n; }

// linear index -> tile coordinate
EXO_HD TileCoord raster_decode(const Raster& r, int64_t t) {
  // "major" = the banded dimension, "minor" = the other one
  const int32_t major = r.along_m ? r.tiles_m : r.tiles_n;
  const int32_t minor = r.along_m ? r.tiles_n : r.tiles_m;
  const int64_t per_band = (int64_t)r.band * minor;
  const int32_t b = (int32_t)(t / per_band);
  const int64_t in_band = t - (int64_t)b * per_band;
  const int32_t first = b * r.band;
  const int32_t width = (major - first) < r.band ? (major - first) : r.band;  // last band may be narrower
  const int32_t i_minor = (int32_t)(in_band / width);
  const int32_t i_major = first + (int32_t)(in_band - (int64_t)i_minor * width);
  TileCoord c;
  c.m = r.along_m ? i_major : i_minor;
  c.n = r.along_m ? i_minor : i_major;
  return c;
}

}  // namespace exo
