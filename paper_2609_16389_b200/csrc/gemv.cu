// fp32 GEMV, y = alpha*A*x + beta*y, for a row- or column-major A: a memory-bound companion of the GEMM.
//
// The paper's second evaluation workload (Section 6) is a full-precision fp32 GEMV built from warp
// shuffles and scalar math, with the roofline 2 FLOP per 4 bytes of matrix read.  The same structure
// is used here: one warp per row, 128-bit coalesced loads along the row, a shuffle tree, one store.
// No tensor cores: the bound is HBM bandwidth, so what matters is enough bytes in flight per SM and
// a grid that is a multiple of the SM count.
#include <cooperative_groups.h>
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

// Column-major A (M contiguous): a lane owns V consecutive rows, so a warp's load of one column is
// contiguous (512 bytes for V == 4).  The columns are split twice: over the CTAs of a thread-block
// cluster, and inside a CTA over its eight warps (warp w takes every eighth column), which gives the
// occupancy a bandwidth-bound kernel needs without relying on deep per-thread unrolling.  Partial sums
// meet in shared memory (warps, in warp order) and then in distributed shared memory (CTAs, in rank
// order): fixed orders, so the result does not depend on timing.
// V == 4: 128-bit loads (lda % 4 == 0, A 16-byte aligned).
constexpr int kColThreads = 256;
constexpr int kColWarps = kColThreads / 32;

template <int V>
__global__ void __launch_bounds__(kColThreads)
exo_gemv_colmajor_kernel(int64_t M, int64_t N, const float* __restrict__ A, int64_t lda,
                         const float* __restrict__ x, float* __restrict__ y, float alpha, float beta) {
  namespace cg = cooperative_groups;
  constexpr int ROWS = 32 * V;                   // rows of y per cluster
  __shared__ float part[kColWarps][ROWS];
  __shared__ float red[ROWS];
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned S = cluster.num_blocks(), r = cluster.block_rank();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int64_t row_block = blockIdx.x / S;
  const int64_t row0 = row_block * ROWS + (int64_t)lane * V;
  const int64_t c0 = (N * (int64_t)r) / S, c1 = (N * (int64_t)(r + 1)) / S;   // this CTA's columns
  float acc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) acc[v] = 0.f;
  if (row0 + V <= M) {
    const float* a = A + row0;
    int64_t j = c0 + w;
    for (; j + 3 * kColWarps < c1; j += 4 * kColWarps) {   // four columns in flight per warp
      const float x0 = __ldg(x + j), x1 = __ldg(x + j + kColWarps), x2 = __ldg(x + j + 2 * kColWarps),
                  x3 = __ldg(x + j + 3 * kColWarps);
      if constexpr (V == 4) {
        const float4 a0 = __ldcs(reinterpret_cast<const float4*>(a + j * lda));
        const float4 a1 = __ldcs(reinterpret_cast<const float4*>(a + (j + kColWarps) * lda));
        const float4 a2 = __ldcs(reinterpret_cast<const float4*>(a + (j + 2 * kColWarps) * lda));
        const float4 a3 = __ldcs(reinterpret_cast<const float4*>(a + (j + 3 * kColWarps) * lda));
        acc[0] += (a0.x * x0 + a1.x * x1) + (a2.x * x2 + a3.x * x3);
        acc[1] += (a0.y * x0 + a1.y * x1) + (a2.y * x2 + a3.y * x3);
        acc[2] += (a0.z * x0 + a1.z * x1) + (a2.z * x2 + a3.z * x3);
        acc[3] += (a0.w * x0 + a1.w * x1) + (a2.w * x2 + a3.w * x3);
      } else {
        const float a0 = __ldcs(a + j * lda), a1 = __ldcs(a + (j + kColWarps) * lda),
                    a2 = __ldcs(a + (j + 2 * kColWarps) * lda), a3 = __ldcs(a + (j + 3 * kColWarps) * lda);
        acc[0] += (a0 * x0 + a1 * x1) + (a2 * x2 + a3 * x3);
      }
    }
    for (; j < c1; j += kColWarps) {
      const float xj = __ldg(x + j);
#pragma unroll
      for (int v = 0; v < V; ++v) acc[v] = fmaf(a[j * lda + v], xj, acc[v]);
    }
  } else {   // the last, ragged group of rows
    for (int64_t j = c0 + w; j < c1; j += kColWarps) {
      const float xj = __ldg(x + j);
#pragma unroll
      for (int v = 0; v < V; ++v)
        if (row0 + v < M) acc[v] = fmaf(A[row0 + v + j * lda], xj, acc[v]);
    }
  }
#pragma unroll
  for (int v = 0; v < V; ++v) part[w][lane * V + v] = acc[v];
  __syncthreads();
  if (threadIdx.x < ROWS) {   // the eight warps' sums, in warp order
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < kColWarps; ++q) sum += part[q][threadIdx.x];
    red[threadIdx.x] = sum;
  }
  cluster.sync();
  // CTA r finishes rows [r * ROWS / S, (r + 1) * ROWS / S) of the cluster's block, adding in rank order
  const int per = ROWS / (int)S;
  if ((int)threadIdx.x < per) {
    const int local = (int)r * per + (int)threadIdx.x;
    float sum = 0.f;
    for (unsigned q = 0; q < S; ++q) sum += cluster.map_shared_rank(red, q)[local];
    const int64_t row = row_block * ROWS + local;
    if (row < M) y[row] = beta != 0.f ? fmaf(beta, y[row], alpha * sum) : alpha * sum;
  }
  cluster.sync();   // no CTA leaves while a peer may still read its sums
}

}  // namespace

extern "C" exo_gemm_status_t exo_gemv_run_colmajor(int64_t M, int64_t N, const float* A, int64_t lda, const float* x,
                                                   float* y, float alpha, float beta, void* cuda_stream) {
  if (M < 0 || N < 0 || lda < (M > 1 ? M : 1)) return EXO_GEMM_ERR_INVALID_ARG;
  if (M == 0) return EXO_GEMM_OK;
  if (!y || (N > 0 && alpha != 0.f && (!A || !x))) return EXO_GEMM_ERR_NULL;
  int device = 0, major = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return EXO_GEMM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return EXO_GEMM_ERR_CUDA;
  if (major != 10) return EXO_GEMM_ERR_ARCH;
  const int64_t n_eff = alpha != 0.f ? N : 0;  // alpha == 0: A and x are not read
  const bool vec = (lda % 4 == 0) && ((uintptr_t)A & 15u) == 0 && M >= 128;
  const int rows = 32 * (vec ? 4 : 1);
  const int64_t row_blocks = (M + rows - 1) / rows;
  unsigned S = 8;                              // portable cluster size; fewer when there are few columns
  while (S > 1 && n_eff < 4 * kColWarps * (int64_t)S) S >>= 1;
  if (row_blocks * S >= (1LL << 31)) return EXO_GEMM_ERR_UNSUPPORTED;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)(row_blocks * S), 1, 1);
  lc.blockDim = dim3(kColThreads, 1, 1);
  lc.stream = (cudaStream_t)cuda_stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = S;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  cudaError_t e = vec ? cudaLaunchKernelEx(&lc, exo_gemv_colmajor_kernel<4>, M, n_eff, A, lda, x, y, alpha, beta)
                      : cudaLaunchKernelEx(&lc, exo_gemv_colmajor_kernel<1>, M, n_eff, A, lda, x, y, alpha, beta);
  return e == cudaSuccess ? EXO_GEMM_OK : EXO_GEMM_ERR_CUDA;
}

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
