// Kernel parameter block and compile-time geometry shared by the host plan and
// the device kernel.
#pragma once
#include <stdint.h>

#include "tile_scheduler.h"

namespace exo {

constexpr int kBlockM = 128;        // rows of C per CTA (one TMEM lane per row)
constexpr int kBlockK = 64;         // 16-bit elements of K per sub-block: 128 bytes = one swizzle span
constexpr int kUmmaK = 16;          // K of one tcgen05.mma for 16-bit inputs (32 bytes; 8 for tf32)
// warp 0 producer of A, warp 1 MMA issuer + TMEM owner, warps 2..9 epilogue, warp 10 producer of B
constexpr int kNumThreads = 352;
constexpr int kProducerBWarp = 10;
constexpr int kEpiWarps = 8;        // two per TMEM lane quadrant, each taking every other column chunk
constexpr int kEpiBufBytes = 4096;  // one staging buffer: 32 rows x 128 bytes
constexpr int kMaxEpiBufs = 2;      // staging buffers per epilogue warp: 1 or 2 (chosen per plan)
constexpr int kMaxStages = 8;
constexpr int kSmemLimit = 232448;  // 227 KB opt-in limit per CTA
constexpr int kBarrierBytes = 512;
constexpr int kATileBytes = kBlockM * kBlockK * 2;  // 16 KB

// Bytes of one pipeline stage in one CTA: its A rows plus its share of B.
#if defined(__CUDACC__)
#define EXO_CX __host__ __device__ constexpr
#else
#define EXO_CX constexpr
#endif
// A stage holds `ksub` sub-blocks of 64 k-elements (1 or 2): one barrier round trip per stage.
// `mrep` = 128-row blocks of A per CTA (1, or 2 for the tall tile whose two accumulators fill TMEM).
EXO_CX int stage_bytes(int cta_group, int bn, int ksub, int mrep = 1) {
  return ksub * (mrep * kATileBytes + (bn / cta_group) * kBlockK * 2);
}

// Stages that fit beside `epi_bufs` staging buffers per epilogue warp.
EXO_CX int max_stages(int cta_group, int bn, int ksub, int epi_bufs, int mrep = 1) {
  const int n = (kSmemLimit - 1024 /*alignment slack*/ - kBarrierBytes - kEpiWarps * epi_bufs * kEpiBufBytes) /
                stage_bytes(cta_group, bn, ksub, mrep);
  return n > kMaxStages ? kMaxStages : n;
}

// The one-tile-per-CTA kernel (lean_kernel.cuh): 1-CTA tiles of 128 x bn, bn = 64 or 128.
// epilogue warps of a lean tile: one per TMEM lane quadrant and per half of the column chunks
EXO_CX int lean_epi_warps(int bn, int c_bytes) { return (bn * c_bytes / 128) >= 2 ? 8 : 4; }
EXO_CX int lean_threads(int bn, int c_bytes) { return 64 + 32 * lean_epi_warps(bn, c_bytes); }
// the peers' partial sums of the rows a CTA finishes when `split` CTAs (a cluster of 1, 2 or 4) share a tile's K loop
EXO_CX int lean_recv_bytes(int bn, int split) { return split > 1 ? (split - 1) * (4 / split) * (bn / 32) * kEpiBufBytes : 0; }
// shared memory of a lean CTA: the operand ring, one staging buffer per column chunk and quadrant,
// the receive buffer, barriers, alignment slack
EXO_CX int lean_smem_bytes(int bn, int ksub, int stages, int c_bytes, int split) {
  return stages * stage_bytes(1, bn, ksub) + 4 * (bn * c_bytes / 128) * kEpiBufBytes + lean_recv_bytes(bn, split) + kBarrierBytes + 1024;
}
EXO_CX int lean_max_stages(int bn, int ksub, int c_bytes, int split) {
  const int n = (kSmemLimit - 1024 - kBarrierBytes - 4 * (bn * c_bytes / 128) * kEpiBufBytes - lean_recv_bytes(bn, split)) /
                stage_bytes(1, bn, ksub);
  return n > kMaxStages ? kMaxStages : n;
}

// The same for a pair of CTAs per 256 x bn tile (lean_pair_kernel.cuh), bn = 128 or 256: the ring doubles as the
// epilogue's staging area (128 rows x bn of C per CTA) once the accumulator is complete.
EXO_CX int lean_pair_ring_bytes(int bn, int ksub, int stages, int c_bytes) {
  return stages * stage_bytes(2, bn, ksub) > kBlockM * bn * c_bytes ? stages * stage_bytes(2, bn, ksub) : kBlockM * bn * c_bytes;
}
EXO_CX int lean_pair_smem_bytes(int bn, int ksub, int stages, int c_bytes) {
  return lean_pair_ring_bytes(bn, ksub, stages, c_bytes) + kBarrierBytes + 1024;
}
EXO_CX int lean_pair_max_stages(int bn, int ksub) {
  const int n = (kSmemLimit - 1024 - kBarrierBytes) / stage_bytes(2, bn, ksub);
  return n > kMaxStages ? kMaxStages : n;
}
constexpr int kLeanPairThreads = 320;   // producer, MMA issuer, eight epilogue warps

// How one operand is staged.  K-major: per 64-k sub-block one TMA box {64 k, rows},
// sub-blocks rows*128 bytes apart.  MN-major: rows/64 boxes {64 mn, 64*ksub k}.
struct OperandStaging {
  uint32_t mn_major;   // 0: K contiguous in memory, 1: M/N contiguous
  uint32_t desc_hi;    // upper half of the UMMA shared-memory descriptor
  uint32_t lbo_enc;    // leading byte offset >> 4
  uint32_t k_step_enc; // descriptor start-address increment per UMMA_K inside a sub-block (bytes >> 4)
  uint32_t k_sub_enc;  // descriptor start-address increment per 64-k sub-block (bytes >> 4)
};

enum StatusCode : uint32_t {
  kStatusOk = 0,
  kStatusTimeout = 1,
};

enum WaitRole : uint32_t {
  kRoleProducer = 1,
  kRoleMma = 2,
  kRoleEpilogue = 3,
  kRoleProducerTail = 4,
  kRoleEpilogueCin = 5,
  kRoleEpiloguePartials = 6,
};

struct GemmParams {
  int32_t M, N, K;          // canonical problem (C row-major; operands possibly swapped)
  int32_t num_k_blocks;     // ceil(K / (64 * ksub)), or 0 when alpha == 0 / K == 0
  uint32_t sub_k;           // k-elements per sub-block: 64 (16-bit operands) or 32 (fp32 storage, tf32 math)
  uint32_t umma_k;          // k-elements per MMA: 16 or 8
  uint32_t tf32;            // 1: operands are fp32 in memory and multiplied as tf32
  int32_t stages;           // depth of the operand ring (2 .. kMaxStages)
  int32_t epi_bufs;         // staging buffers per epilogue warp: 1 or 2, or 0 = C is stored straight from registers
  Raster raster;
  uint32_t batch;           // matrices in the strided batch (1 = a plain GEMM, 2-D tensor maps)
  uint32_t tiles_per_batch; // raster.tiles_m * raster.tiles_n
  FastDiv by_tiles_per_batch;
  uint32_t a_z_mask, b_z_mask;  // all ones, or 0 for an operand that every matrix of the batch shares
  float alpha, beta;
  uint32_t idesc;           // tcgen05 instruction descriptor
  OperandStaging a, b;
  WorkPlan work;            // whole-K tiles round-robin, then the tail tiles cut along K
  float* split_ws;          // device: fp32 partial accumulators of the slices 1.. of every tail tile
  uint32_t* split_flags;    // device: per tail tile {arrivals of contributing warps, owner warps done}; both only grow
  uint32_t c_evict_first;   // 1: the stores of C carry the L2 evict-first priority
  uint32_t reduce_add;      // 1: the parts of a cut tile add onto C (TMA reduce) instead of meeting in the workspace
  uint32_t split_arrivals;  // arrivals per contributing part of a tile and run: its epilogue warps (x accumulators)
  void* c_ptr;              // C of matrix 0 and its strides in bytes (read by the direct stores only)
  int64_t ldc_bytes, c_batch_bytes;
  uint32_t* status;         // device: 8 words {code, role, barrier, tile, k_block, cta, -, -}
  uint64_t timeout_cycles;  // bound of every device-side wait, in SM clocks
  int64_t debug_skip_k_block;  // -1, or the producer k-block of CTA 0 whose loads are skipped
};

}  // namespace exo
