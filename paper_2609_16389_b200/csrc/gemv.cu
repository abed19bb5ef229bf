// fp32 GEMV, y = alpha*A*x + beta*y, for a row-major A: a memory-bound companion of the GEMM.
//
// The paper's second evaluation workload (Section 6) is a full-precision fp32 GEMV built from warp
// shuffles and scalar math, with the roofline 2 FLOP per 4 bytes of matrix read.  The same structure
// is used here: one warp per row, 128-bit coalesced loads along the row, a shuffle tree, one store.
// No tensor cores: the bound is HBM bandwidth, so what matters is enough bytes in flight per SM and
// a grid that is a multiple of the SM count.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/exo_gemm.h"

namespace {

constexpr int kGemvThreads = 256;   // 8 warps per CTA
constexpr int kGemvCtasPerSm = 8;   // 64 resident warps per SM

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// VEC: A rows and x are 16-byte aligned (lda % 4 == 0): float4 loads, four independent partial sums.
template <bool VEC>
__global__ void __launch_bounds__(kGemvThreads)
exo_gemv_rowmajor_kernel(int64_t M, int64_t N, const float* __restrict__ A, int64_t lda,
                         const float* __restrict__ x, float* __restrict__ y, float alpha, float beta) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * kGemvThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kGemvThreads) >> 5;
  for (int64_t row = warp; row < M; row += nwarps) {
    const float* a = A + row * lda;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int64_t j = 0;
    if (VEC) {
      const float4* a4 = reinterpret_cast<const float4*>(a);
      const float4* x4 = reinterpret_cast<const float4*>(x);
      const int64_t n4 = N >> 2;
      int64_t q = lane;
      for (; q + 96 < n4; q += 128) {  // four 128-bit loads of A in flight per lane
        const float4 v0 = __ldcs(a4 + q), v1 = __ldcs(a4 + q + 32), v2 = __ldcs(a4 + q + 64), v3 = __ldcs(a4 + q + 96);
        const float4 w0 = __ldg(x4 + q), w1 = __ldg(x4 + q + 32), w2 = __ldg(x4 + q + 64), w3 = __ldg(x4 + q + 96);
        s0 += v0.x * w0.x + v0.y * w0.y + v0.z * w0.z + v0.w * w0.w;
        s1 += v1.x * w1.x + v1.y * w1.y + v1.z * w1.z + v1.w * w1.w;
        s2 += v2.x * w2.x + v2.y * w2.y + v2.z * w2.z + v2.w * w2.w;
        s3 += v3.x * w3.x + v3.y * w3.y + v3.z * w3.z + v3.w * w3.w;
      }
      for (; q < n4; q += 32) {
        const float4 v = __ldcs(a4 + q);
        const float4 w = __ldg(x4 + q);
        s0 += v.x * w.x + v.y * w.y + v.z * w.z + v.w * w.w;
      }
      j = n4 << 2;
    }
    for (int64_t k = j + lane; k < N; k += 32) s1 += a[k] * __ldg(x + k);  // ragged tail, or the unaligned path
    const float sum = warp_sum((s0 + s1) + (s2 + s3));
    if (lane == 0) y[row] = beta != 0.f ? fmaf(beta, y[row], alpha * sum) : alpha * sum;
  }
}

}  // namespace

extern "C" exo_gemm_status_t exo_gemv_run(int64_t M, int64_t N, const float* A, int64_t lda, const float* x,
                                          float* y, float alpha, float beta, void* cuda_stream) {
  if (M < 0 || N < 0 || lda < (N > 1 ? N : 1)) return EXO_GEMM_ERR_INVALID_ARG;
  if (M == 0) return EXO_GEMM_OK;
  if (!y || (N > 0 && alpha != 0.f && (!A || !x))) return EXO_GEMM_ERR_NULL;
  int device = 0, sms = 0, major = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return EXO_GEMM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return EXO_GEMM_ERR_CUDA;
  if (major != 10) return EXO_GEMM_ERR_ARCH;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return EXO_GEMM_ERR_CUDA;
  const int64_t warps_needed = M;
  int64_t ctas = (warps_needed + (kGemvThreads / 32) - 1) / (kGemvThreads / 32);
  const int64_t full = (int64_t)sms * kGemvCtasPerSm;  // a multiple of the SM count
  if (ctas > full) ctas = full;
  const bool vec = (lda % 4 == 0) && (((uintptr_t)A | (uintptr_t)x) & 15u) == 0;
  const int64_t n_eff = alpha != 0.f ? N : 0;  // alpha == 0: A and x are not read
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (vec) exo_gemv_rowmajor_kernel<true><<<(unsigned)ctas, kGemvThreads, 0, st>>>(M, n_eff, A, lda, x, y, alpha, beta);
  else exo_gemv_rowmajor_kernel<false><<<(unsigned)ctas, kGemvThreads, 0, st>>>(M, n_eff, A, lda, x, y, alpha, beta);
  return cudaGetLastError() == cudaSuccess ? EXO_GEMM_OK : EXO_GEMM_ERR_CUDA;
}
