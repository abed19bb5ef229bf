// Copies between a matrix with an arbitrary leading dimension and a plan-owned copy whose rows start on
// 16-byte boundaries.  TMA addresses rows by a byte stride that must be a multiple of 16, so a legal BLAS
// call (the paper's Section 6 measures against BLAS Sgemm) whose leading dimension is not -- an odd number
// of 16-bit elements, say -- cannot be described by a tensor map; such a matrix makes one extra pass
// through these kernels per run (operands before the GEMM, C after it, and before it too if beta != 0).
#pragma once
#include <stdint.h>

namespace exo {

constexpr int kRepackThreads = 256;
constexpr int kRepackPerThread = 8;   // elements of one row per thread

// `outer` rows of `inner` contiguous elements each: dst[o * dst_ld + i] = src[o * src_ld + i].
// One CTA copies a segment of kRepackThreads * kRepackPerThread elements of one row.
template <typename T>
__global__ void __launch_bounds__(kRepackThreads) exo_repack_kernel(T* __restrict__ dst, int64_t dst_ld, const T* __restrict__ src,
                                                                     int64_t src_ld, int64_t inner, uint32_t segments_per_row) {
  const uint32_t row = blockIdx.x / segments_per_row;
  const uint32_t seg = blockIdx.x - row * segments_per_row;
  const T* s = src + (int64_t)row * src_ld;
  T* d = dst + (int64_t)row * dst_ld;
  const int64_t i0 = (int64_t)seg * (kRepackThreads * kRepackPerThread) + threadIdx.x;
#pragma unroll
  for (int k = 0; k < kRepackPerThread; ++k) {
    const int64_t i = i0 + (int64_t)k * kRepackThreads;   // consecutive threads, consecutive elements
    if (i < inner) d[i] = s[i];
  }
}

// Enqueues the copy; false if the matrix has more row segments than a grid can have (then nothing is enqueued).
inline bool repack_grid(int64_t inner, int64_t outer, uint32_t* segments_per_row, uint32_t* blocks) {
  const int64_t per = kRepackThreads * kRepackPerThread;
  const int64_t seg = (inner + per - 1) / per;
  if (seg < 1 || outer < 1 || seg * outer > 2147483647LL) return false;
  *segments_per_row = (uint32_t)seg;
  *blocks = (uint32_t)(seg * outer);
  return true;
}

}  // namespace exo
