// Persistent warp-specialised tcgen05 GEMM kernel for sm_100a.
//
// One CTA (CTA_GROUP == 1) or a pair of CTAs on two SMs (CTA_GROUP == 2, a
// 2-CTA cluster) computes output tiles of (128 * CTA_GROUP) x BN, one after
// another, taken round-robin from a band-swizzled raster.  Roles per CTA:
//
//   warps 0 and 10,    producers: TMA loads of the A (warp 0) and B (warp 10) k-blocks
//   one lane each      into a ring of shared-memory stages (full/empty mbarriers)
//   warp 1, one lane   MMA issuer (leader CTA only): tcgen05.mma from shared
//                      memory into one of two TMEM accumulators; tcgen05.commit
//                      releases stages and publishes finished accumulators
//   warp 1             owns the TMEM allocation
//   warps 2..9         epilogue: tcgen05.ld the accumulator (warp w reads TMEM
//                      lanes 32*(w%4).. and every other 128-byte column chunk),
//                      alpha*acc + beta*C_in in fp32, convert, write a 128B-swizzled
//                      staging buffer, TMA store
//
// The structure follows the kernel class of the paper's Section 6 (persistent,
// warp-specialised, TMA + swizzled shared memory + asynchronous tensor-core
// MMA, 2-CTA clusters), re-designed for Blackwell: the accumulator lives in
// tensor memory instead of registers, one thread issues the MMA, and completion
// is tracked by tcgen05.commit on mbarriers instead of commit groups.  The
// synchronisation rules it obeys are the ones the paper's Section 2.2 bug
// catalogue spells out: a stage is refilled only after the *asynchronous* MMAs
// that read it completed (commit -> empty barrier), an accumulator is read only
// after the MMAs that write it completed (commit -> tmem_full barrier), and a
// release that covers another CTA's shared memory is cluster-scoped.
//
// Every wait is bounded: when one gives up, the kernel records where, all roles
// leave their loops, TMEM is freed and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "gemm_params.h"
#include "ptx.cuh"

namespace exo {

enum OutKind : int { kOutBf16 = 0, kOutFp16 = 1, kOutFp32 = 2 };

// Development aid, compiled only with -DEXO_GEMM_TRACE: CTA 0 stamps clock64() at
// points of its three roles into the words that follow the status block.
#ifdef EXO_GEMM_TRACE
#define EXO_TRACE(role, idx, field, cap)                                                        \
  do {                                                                                          \
    if (blockIdx.x == 0 && (idx) < (cap))                                                       \
      reinterpret_cast<long long*>(p.status + 8)[((role) * 4096 + (idx)) * 2 + (field)] = clock64(); \
  } while (0)
// per-chunk stamps of the first epilogue warp: k = 0 buffer free, 1 accumulator in registers, 2 converted
// and staged (or stored), 3 store issued
#define EXO_TRACE_CHUNK(gc, k)                                                                 \
  do {                                                                                          \
    if (warp == 2 && lane == 0) EXO_TRACE(1, 2048 + 4 * (gc) + (k), 0, 4090);                   \
  } while (0)
// stamps of the first epilogue warp between two tiles: k = 0 .. 7 per work item
#define EXO_TRACE_TILE(it, k)                                                                  \
  do {                                                                                          \
    if (warp == 2 && lane == 0) EXO_TRACE(0, 2048 + 8 * (it) + (k), 0, 4090);                   \
  } while (0)
#else
#define EXO_TRACE(role, idx, field, cap) do {} while (0)
#define EXO_TRACE_CHUNK(gc, k) do {} while (0)
#define EXO_TRACE_TILE(it, k) do {} while (0)
#endif

struct WaitSite {
  uint32_t role, barrier, tile, k_block;
};

template <bool CLUSTER>
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const GemmParams& p, WaitSite site) {
  const long long t0 = clock64();
  uint32_t n = 0;
  for (;;) {
    const bool done = CLUSTER ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity);
    if (done) return true;
    if ((++n & 63u) == 0u) {
      if (*(volatile uint32_t*)p.status != kStatusOk) return false;  // another role gave up
      if ((uint64_t)(clock64() - t0) > p.timeout_cycles) {
        if (atomicCAS(p.status, (uint32_t)kStatusOk, (uint32_t)kStatusTimeout) == kStatusOk) {
          p.status[1] = site.role;
          p.status[2] = site.barrier;
          p.status[3] = site.tile;
          p.status[4] = site.k_block;
          p.status[5] = blockIdx.x;
          __threadfence();
        }
        return false;
      }
    }
  }
}

// Bounded mbarrier wait.  Returns false if the wait was abandoned.
template <bool CLUSTER>
__device__ __forceinline__ bool wait_barrier(uint32_t bar, uint32_t parity, const GemmParams& p,
                                             WaitSite site) {
#pragma unroll 1
  for (int i = 0; i < 8; ++i) {
    const bool done = CLUSTER ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity);
    if (done) return true;
  }
  return wait_slow<CLUSTER>(bar, parity, p, site);
}

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, const OperandStaging& op) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (op.lbo_enc << 16);
  return ((uint64_t)op.desc_hi << 32) | lo;
}

template <int OUT>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  if constexpr (OUT == kOutBf16) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
  } else {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
  }
}

template <int OUT>
__device__ __forceinline__ float2 unpack2(uint32_t w) {
  if constexpr (OUT == kOutBf16) {
    return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w));
  } else {
    return __half22float2(*reinterpret_cast<__half2*>(&w));
  }
}

// Default policy: a CTA group loads all of its own operands.  The alternative (a cluster of two
// CTA pairs that split the loads of the A rows they have in common) supplies kPairs == 2 and the
// load functions for the shared half-blocks; it lives in a translation unit of its own.
struct NoShare {
  static constexpr int kPairs = 1;
};

// MREP = 128-row blocks of C per CTA.  1: the two TMEM accumulators alternate between consecutive
// tiles, so a tile's epilogue overlaps the next tile's main loop.  2 (the "tall" tile, 256 x BN per
// CTA): both accumulators belong to one tile -- A_lo and A_hi are multiplied with the same B block, so
// a quarter less operand data enters shared memory per flop -- and the epilogue is exposed.
// REDUCE: the kernel can add the parts of a cut tile onto C (p.reduce_add); compiled only into the few
// instantiations that plans with that flag use -- the extra paths cost the others 1-2 % where the epilogue
// bounds a tile.
template <int CTA_GROUP, int BN, int OUT, int KSUB, class Share = NoShare, int MREP = 1, bool REDUCE = false>
__global__ void __launch_bounds__(kNumThreads, 1)
exo_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
  const int32_t STAGE_K = (int32_t)p.sub_k * KSUB;   // k-elements per stage (64 or 32 per sub-block)
  constexpr int B_ROWS = BN / CTA_GROUP;             // rows of the B tile this CTA stages
  constexpr int STAGE_BYTES = stage_bytes(CTA_GROUP, BN, KSUB, MREP);
  constexpr int A_BYTES = KSUB * kATileBytes * MREP; // the A part of a stage
  constexpr int CTA_M = kBlockM * MREP;              // rows of C per CTA
  static_assert(!REDUCE || (OUT == kOutFp32 && MREP == 1 && Share::kPairs == 1), "reduce-add: fp32 C, plain tiles");
  static_assert(MREP == 1 || (MREP == 2 && CTA_GROUP == 2 && BN == 256 && KSUB == 1 && Share::kPairs == 1),
                "the tall tile exists for 2-CTA 256-column tiles only");
  constexpr uint32_t TMEM_COLS = 2 * BN;             // two accumulators; 128, 256 or 512 columns
  constexpr int CW = (OUT == kOutFp32) ? 32 : 64;    // columns per epilogue chunk = 128 bytes of C
  constexpr int NCHUNK = BN / CW;
  constexpr bool PAIR = CTA_GROUP == 2;
  constexpr int NPAIR = Share::kPairs;              // CTA pairs per cluster that compute side by side in N
  constexpr bool SHARE = NPAIR > 1;                  // ... and fetch half of their common A rows each
  constexpr int CLUSTER = CTA_GROUP * NPAIR;
  static_assert(!SHARE || (PAIR && NPAIR == 2), "operand sharing is built on CTA pairs");
  static_assert(BN == 64 || BN == 128 || BN == 256, "tile N");
  const uint32_t STAGES = (uint32_t)p.stages;         // ring depth, chosen by the host plan
  const uint32_t EPI_BUFS = (uint32_t)p.epi_bufs;     // staging buffers per epilogue warp (1 or 2)

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms are 1 KB
  const uint32_t stage0 = smem_base;
  const uint32_t epi0 = smem_base + STAGES * STAGE_BYTES;
  const uint32_t bar0 = epi0 + kEpiWarps * EPI_BUFS * kEpiBufBytes;
  auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](uint32_t a) { return bar0 + 8u * (2 * kMaxStages + a); };
  auto tempty_bar = [&](uint32_t a) { return bar0 + 8u * (2 * kMaxStages + 2 + a); };
  auto cin_bar = [&](uint32_t w, uint32_t b) { return bar0 + 8u * (2 * kMaxStages + 4 + kMaxEpiBufs * w + b); };
  // "the accumulator of the owning slice holds the other slices' sum": used at most once per launch
  const uint32_t tfilled_bar = bar0 + 8u * (2 * kMaxStages + 4 + kMaxEpiBufs * kEpiWarps);
  const uint32_t tmem_slot = tfilled_bar + 8u;
  static_assert(8 * (2 * kMaxStages + 5 + kMaxEpiBufs * kEpiWarps) + 4 <= kBarrierBytes, "barrier area");

  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t cluster_rank = PAIR ? ptx::cluster_ctarank() : 0u;
  const uint32_t cta_rank = cluster_rank & 1u;            // position inside the CTA pair
  const uint32_t leader = cluster_rank & ~1u;             // cluster rank of this pair's MMA-issuing CTA
  // With operand sharing the grid is cut into slots of four CTAs.  The launch asks for 4-CTA clusters
  // but lets the device substitute two 2-CTA clusters where no four SMs of one GPC are free; such a
  // slot computes the same two tiles with each pair loading all of its A rows itself.
  const uint32_t slot_rank = (uint32_t)blockIdx.x & (uint32_t)(CLUSTER - 1);
  const uint32_t pair_id = SHARE ? slot_rank >> 1 : 0u;   // which of the slot's two tiles
  const bool quad = SHARE && ptx::cluster_nctarank() == 4u;
  const int64_t worker = blockIdx.x / CLUSTER;
  const int64_t num_workers = gridDim.x / CLUSTER;
  const int32_t nkb = p.num_k_blocks;
  // From which item index on an owning slice of a tail tile finds the other slices' sum preloaded in
  // its accumulator (see the epilogue role): the partials must have been published and read back while
  // the item before it ran.  Two whole tiles in front always leave that time; a single one does if the
  // K loop is long (measured behind one whole wave: -1.4 % at K = 3072, +1.4 to +2.1 % at 4096, +4 % at
  // 8192).
  const int64_t preload_from = (int64_t)nkb * STAGE_K >= 4096 ? 1 : 2;

  if (threadIdx.x == 0) EXO_TRACE(2, 4095, 0, 4096);
  // ---------------------------------------------------------------- setup
  // An epilogue warp prepares the barriers, a lane each: the producer and MMA warps spend the same time
  // on their first work item (below), whose parameter loads and divisions would otherwise sit between
  // the end of the setup and the first copy.
  if (warp == 2) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tm_a);
      ptx::prefetch_tensormap(&tm_b);
    }
    // the barrier words are consecutive: full[kMaxStages], empty[kMaxStages], tfull[2], tempty[2], C_in, tfilled
    constexpr uint32_t kBarriers = 2 * kMaxStages + 5 + kMaxEpiBufs * kEpiWarps;
    for (uint32_t i = lane; i < kBarriers; i += 32u) {
      uint32_t count = 1;
      if (i >= (uint32_t)kMaxStages && i < 2u * kMaxStages) count = quad ? 2u : 1u;  // every pair whose CTAs fill the stage releases it
      if ((i >= 2u * kMaxStages + 2u && i < 2u * kMaxStages + 4u) || i == kBarriers - 1u) count = kEpiWarps * CTA_GROUP;
      ptx::mbar_init(bar0 + 8u * i, count);
    }
    ptx::fence_mbar_init();
    if (lane == 0) ptx::prefetch_tensormap(&tm_c);
  }
  if (warp == 1) {
    ptx::tmem_alloc<CTA_GROUP>(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish<CTA_GROUP>();
  }
  // Arrive at the cluster barrier as early as possible (a warp's arrival follows its own share of the
  // setup and publishes it) and wait as late as possible: the barrier's latency then overlaps the
  // first work item's arithmetic instead of following it.
  if constexpr (PAIR) ptx::cluster_arrive();
  // The first work item depends on kernel parameters only, so the warps that need it first compute it
  // while the barriers are being set up (the epilogue warps need theirs a whole main loop later).
  const bool batched = p.batch > 1;
  auto tile_coord = [&](int64_t t, uint32_t* bz) {
    *bz = batched ? fast_div((uint32_t)t, p.by_tiles_per_batch) : 0u;  // which matrix of the batch
    return raster_decode(p.raster, batched ? (uint32_t)t - *bz * p.tiles_per_batch : t);
  };
  WorkItem wi_first{};
  TileCoord tc_first{};
  uint32_t bz_first = 0;
  bool have_first = false;
  if (warp < 2 || warp == (uint32_t)kProducerBWarp) {
    have_first = work_item(p.work, worker, num_workers, 0, nkb, &wi_first);
    if (have_first && warp != 1) tc_first = tile_coord(wi_first.tile, &bz_first);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if constexpr (PAIR) ptx::cluster_wait();  // peer barriers and tensor memory exist before anything remote touches them
  ptx::tc_fence_after_sync();
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot) : "memory");

  // Everything above touched only this CTA's shared and tensor memory, so with programmatic
  // dependent launch it overlaps the tail of the previous kernel in the stream.  Each role waits for
  // that kernel itself at the start of its role, with every lane: before that wait no thread reads
  // global memory, the status word included.

  bool ok = true;
  if (threadIdx.x == 0) EXO_TRACE(2, 4094, 0, 4096);

  if (warp == 0 || warp == (uint32_t)kProducerBWarp) {
    // ============================================================ producer
    // Issuing a stage's copies from one lane takes a few hundred clocks, which is what a stage's MMAs
    // take too: two warps share the work (A and the byte count from warp 0, B from the other warp).
    const bool do_a = warp == 0, do_b = warp == (uint32_t)kProducerBWarp;
    // The whole warp runs the loop (uniform control flow); one elected lane issues.
    uint32_t s = 0, ph = 0;
    int64_t issued = 0;
    // in a pair, both CTAs' loads are counted on the leader's full barrier
    const uint32_t full0 = PAIR ? ptx::map_to_cta(full_bar(0), leader) : full_bar(0);
    // The operands may be the previous kernel's output, and the status word that the bounded waits poll
    // may still be about to be cleared by the work before this kernel: every lane waits for it here.  (The
    // first wait of the loop below passes at once, so this is as late as a wait before the first copy.)
    ptx::grid_dependency_wait();
    for (int64_t it = 0; ok; ++it) {
      WorkItem wi = wi_first;
      TileCoord tc = tc_first;
      uint32_t bz = bz_first;
      if (it == 0) {
        if (!have_first) break;
      } else {
        if (!work_item(p.work, worker, num_workers, it, nkb, &wi)) break;
        tc = tile_coord(wi.tile, &bz);
      }
      const int64_t t = wi.tile;
      const int32_t a_mn0 = tc.m * (CTA_M * CTA_GROUP) + (int32_t)cta_rank * CTA_M;
      const int32_t b_mn0 = (tc.n * NPAIR + (int32_t)pair_id) * BN + (int32_t)cta_rank * B_ROWS;
      for (int32_t kb = wi.kb_begin; kb < wi.kb_end; ++kb) {
        ok = wait_barrier<PAIR>(empty_bar(s), ph ^ 1u, p, WaitSite{kRoleProducer, s, (uint32_t)t, (uint32_t)kb});
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const bool skip = (p.debug_skip_k_block == issued) && blockIdx.x == 0;
        if (ptx::elect_one()) {
          EXO_TRACE(0, issued, 0, 4096);
          if (cta_rank == 0 && do_a) ptx::mbar_arrive_expect_tx(full_bar(s), STAGE_BYTES * CTA_GROUP);
          if (!skip) {
            const uint32_t a_dst = stage0 + s * STAGE_BYTES;
            const uint32_t b_dst = a_dst + A_BYTES;
            const uint32_t bar = full0 + 8u * s;
            const int32_t k0 = kb * STAGE_K;
            // This loop runs once per stage in a single lane and can bound the whole pipeline when a stage's
            // MMAs are short: box counts and offsets are compile-time constants and the batched / plain
            // distinction is taken once per stage, not once per copy.
            constexpr int A_BOXES = CTA_M / 64, B_BOXES = B_ROWS / 64;   // M/N-contiguous 16-bit operands: 64 per box
            constexpr uint32_t MN_BOX_BYTES = KSUB * 8192u;             // one box: 64 * KSUB k-rows of 128 bytes
            auto stage_loads = [&](auto&& load) {
              if (!do_a) {
              } else if (quad) {
                if constexpr (SHARE) {
                  // The other pair's CTA of the same rank needs the same 128 rows of A: each of the two
                  // fetches 64 of them and the copy lands in both CTAs' stages; each copy's bytes count
                  // on the full barrier of the receiving CTA's own pair leader.
                  const uint16_t both = (uint16_t)((1u << cta_rank) | (1u << (cta_rank + 2u)));
                  auto load_shared = [&](uint32_t dst, int32_t x, int32_t y) {
                    if (batched) Share::load_3d(dst, &tm_a, x, y, (int32_t)(bz & p.a_z_mask), bar, both);
                    else Share::load_2d(dst, &tm_a, x, y, bar, both);
                  };
                  if (!p.a.mn_major) {
#pragma unroll
                    for (int h = 0; h < KSUB; ++h)
                      load_shared(a_dst + h * kATileBytes + pair_id * (kATileBytes / 2), k0 + h * (int32_t)p.sub_k,
                                  a_mn0 + (int32_t)pair_id * (kBlockM / 2));
                  } else if (!p.tf32) {  // two boxes of 64 rows: one each
                    load_shared(a_dst + pair_id * MN_BOX_BYTES, a_mn0 + 64 * (int32_t)pair_id, k0);
                  } else {               // fp32 storage: four boxes of 32 rows, two each
#pragma unroll
                    for (int b = 0; b < 2; ++b)
                      load_shared(a_dst + (2 * pair_id + b) * (MN_BOX_BYTES / 2), a_mn0 + 32 * (int32_t)(2 * pair_id + b), k0);
                  }
                }
              } else if (SHARE && !p.a.mn_major) {  // substituted pair: both 64-row halves, same tensor map
#pragma unroll
                for (int h = 0; h < KSUB; ++h) {
                  load(a_dst + h * kATileBytes, &tm_a, k0 + h * (int32_t)p.sub_k, a_mn0);
                  load(a_dst + h * kATileBytes + kATileBytes / 2, &tm_a, k0 + h * (int32_t)p.sub_k, a_mn0 + kBlockM / 2);
                }
              } else if (!p.a.mn_major) {
#pragma unroll
                for (int h = 0; h < KSUB; ++h) load(a_dst + h * (kATileBytes * MREP), &tm_a, k0 + h * (int32_t)p.sub_k, a_mn0);
              } else if (!p.tf32) {
#pragma unroll
                for (int b = 0; b < A_BOXES; ++b) load(a_dst + b * MN_BOX_BYTES, &tm_a, a_mn0 + 64 * b, k0);
              } else {  // fp32 storage: 32 elements per 128 bytes, twice as many boxes of half the size
#pragma unroll
                for (int b = 0; b < 2 * A_BOXES; ++b) load(a_dst + b * (MN_BOX_BYTES / 2), &tm_a, a_mn0 + 32 * b, k0);
              }
              if (!do_b) {
              } else if (!p.b.mn_major) {
#pragma unroll
                for (int h = 0; h < KSUB; ++h) load(b_dst + h * (B_ROWS * 128), &tm_b, k0 + h * (int32_t)p.sub_k, b_mn0);
              } else if (!p.tf32) {
#pragma unroll
                for (int b = 0; b < B_BOXES; ++b) load(b_dst + b * MN_BOX_BYTES, &tm_b, b_mn0 + 64 * b, k0);
              } else {
#pragma unroll
                for (int b = 0; b < 2 * B_BOXES; ++b) load(b_dst + b * (MN_BOX_BYTES / 2), &tm_b, b_mn0 + 32 * b, k0);
              }
            };
            if (!batched) {
              stage_loads([&](uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y) {
                if constexpr (PAIR) ptx::tma_load_2d_pair(dst, map, x, y, bar);
                else ptx::tma_load_2d(dst, map, x, y, bar);
              });
            } else {
              stage_loads([&](uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y) {
                const int32_t z = (int32_t)(bz & (map == &tm_a ? p.a_z_mask : p.b_z_mask));
                if constexpr (PAIR) ptx::tma_load_3d_pair(dst, map, x, y, z, bar);
                else ptx::tma_load_3d(dst, map, x, y, z, bar);
              });
            }
          }
          EXO_TRACE(0, issued, 1, 4096);
        }
        ++issued;
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
    // Tail: do not leave while stage releases addressed to this CTA are still in flight.
    for (uint32_t i = 0; i < STAGES && ok; ++i) {
      ok = wait_barrier<PAIR>(empty_bar(s), ph ^ 1u, p, WaitSite{kRoleProducerTail, s, 0, 0});
      ok = __all_sync(0xffffffffu, ok);
      if (++s == STAGES) { s = 0; ph ^= 1u; }
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer
    if (cta_rank == 0 && nkb > 0) {
      // This warp touches no user memory, but its bounded waits poll the status word, which the work in
      // front of this kernel may still be about to clear; its first real wait is for data that the
      // producers fetch after the same dependency, so this costs no time.
      ptx::grid_dependency_wait();
      uint32_t s = 0, ph = 0, acc = 0, acc_ph = 0;
      const uint16_t kStageMask = quad ? 0xF : (PAIR ? 3 : 1);  // a stage is released in every CTA that fills it
      const uint16_t pair_mask = (uint16_t)((PAIR ? 3u : 1u) << leader);   // the accumulator belongs to this pair
      [[maybe_unused]] int64_t consumed = 0;
      const uint32_t a_step = p.a.k_step_enc, b_step = p.b.k_step_enc;
      const uint32_t a_sub = p.a.k_sub_enc, b_sub = p.b.k_sub_enc;
      constexpr int kMmaPerStage = 4 * KSUB;  // an MMA consumes 32 bytes of K whatever the element size
      const bool tf32 = p.tf32 != 0;
      const int32_t umma_k = (int32_t)p.umma_k;
      auto k_off = [](int32_t k, uint32_t step, uint32_t sub) {  // descriptor offset of the k-th MMA of a stage
        return (uint64_t)((uint32_t)(k & 3) * step + (uint32_t)(k >> 2) * sub);
      };
      const uint32_t idesc = p.idesc;
      // the MMAs of one 128-row block of one stage (elected lane only)
      auto issue_stage = [&](uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, bool first_kb, int32_t k_left) {
        if (k_left >= STAGE_K && !tf32) {
#pragma unroll
          for (int32_t k = 0; k < kMmaPerStage; ++k)
            ptx::umma_f16<CTA_GROUP>(d_tmem, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub),
                                     idesc, (!first_kb || k != 0) ? 1u : 0u);
        } else if (k_left >= STAGE_K) {
#pragma unroll
          for (int32_t k = 0; k < kMmaPerStage; ++k)
            ptx::umma_tf32<CTA_GROUP>(d_tmem, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub),
                                      idesc, (!first_kb || k != 0) ? 1u : 0u);
        } else {  // ragged last k-block: skip the MMAs that would only read zero fill
          const int32_t n_mma = (k_left + umma_k - 1) / umma_k;
          for (int32_t k = 0; k < n_mma; ++k) {
            const uint32_t accumulate = (!first_kb || k != 0) ? 1u : 0u;
            if (tf32)
              ptx::umma_tf32<CTA_GROUP>(d_tmem, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub),
                                        idesc, accumulate);
            else
              ptx::umma_f16<CTA_GROUP>(d_tmem, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub),
                                       idesc, accumulate);
          }
        }
      };
      for (int64_t it = 0; ok; ++it) {
        WorkItem wi = wi_first;
        if (it == 0) {
          if (!have_first) break;
        } else if (!work_item(p.work, worker, num_workers, it, nkb, &wi)) {
          break;
        }
        const int64_t t = wi.tile;
        // The owning slice of a tail tile that follows at least two whole tiles starts from an accumulator
        // into which the epilogue warps have already written the other slices' partial sums.
        const bool preloaded = MREP == 1 && wi.slices > 1 && wi.slice == 0 && wi.after_whole && it >= preload_from && !(REDUCE && p.reduce_add);
        if constexpr (MREP == 1) {
          // the epilogue (of both CTAs) must have drained this accumulator
          ok = wait_barrier<PAIR>(tempty_bar(acc), acc_ph ^ 1u, p, WaitSite{kRoleMma, 100 + acc, (uint32_t)t, 0});
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (preloaded) {  // ... and have filled it again (a barrier of its own: this happens once per launch)
            ok = wait_barrier<PAIR>(tfilled_bar, 0u, p, WaitSite{kRoleMma, 110 + acc, (uint32_t)t, 0});
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          ptx::tc_fence_after_sync();
        }
        for (int32_t kb = wi.kb_begin; kb < wi.kb_end; ++kb) {
          ok = wait_barrier<PAIR>(full_bar(s), ph, p, WaitSite{kRoleMma, s, (uint32_t)t, (uint32_t)kb});
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t a_addr = stage0 + s * STAGE_BYTES;
          const uint64_t a_desc = make_smem_desc(a_addr, p.a);
          const uint64_t b_desc = make_smem_desc(a_addr + A_BYTES, p.b);
          const int32_t k_left = p.K - kb * STAGE_K;
          const bool first_kb = kb == wi.kb_begin, last_kb = kb == wi.kb_end - 1;
#pragma unroll
          for (uint32_t r = 0; r < (uint32_t)MREP; ++r) {
            // tall tile: accumulator r holds rows 128r.. of the CTA's block; the previous tile's epilogue
            // drains accumulator 0 first, so this tile's first MMAs overlap the draining of accumulator 1
            const uint32_t a_acc = MREP == 1 ? acc : r;
            if (MREP == 2 && first_kb) {
              ok = wait_barrier<PAIR>(tempty_bar(a_acc), acc_ph ^ 1u, p, WaitSite{kRoleMma, 100 + a_acc, (uint32_t)t, 0});
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              ptx::tc_fence_after_sync();
            }
            if (ptx::elect_one()) {  // the same lane every time: commits track this thread's MMAs
              if (r == 0) EXO_TRACE(1, consumed, 0, 4096);
              // the second 128-row block of A lies 16 KB after the first in every staging layout
              issue_stage(tmem_base + a_acc * BN, a_desc + (uint64_t)(r * (kATileBytes >> 4)), b_desc, first_kb && !preloaded, k_left);
              if (r == MREP - 1) ptx::umma_commit<CTA_GROUP>(empty_bar(s), kStageMask);  // stage free once these MMAs completed
              if (last_kb) ptx::umma_commit<CTA_GROUP>(tfull_bar(a_acc), pair_mask);      // accumulator complete
              if (r == MREP - 1) EXO_TRACE(1, consumed, 1, 4096);
            }
          }
          if (!ok) break;
          ++consumed;
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if (MREP == 2 || (acc ^= 1u) == 0u) acc_ph ^= 1u;
      }
    }
  } else {
    // ============================================================ epilogue
    // Warp w reads TMEM lanes 32*(w%4)..+31 (a hardware rule) and, of the tile's column
    // chunks (128 bytes of C per row each), the left (half == 0) or the right half.
    constexpr int UPC = CW / 32;                       // 32-column TMEM loads per chunk
    constexpr int kHalfChunks = (NCHUNK + 1) / 2;      // chunks per warp of a lane quadrant
    constexpr uint32_t kOwnerWarps = kEpiWarps * CTA_GROUP;   // epilogue warps of the CTA group that owns a tile
    // this warp is done with the partial sums of tail tile `ti` (see wait_partials)
    auto partials_consumed = [&](int32_t ti) {
      __syncwarp();
      if (ptx::elect_one()) ptx::red_release_gpu_add(p.split_flags + 2 * (ti * NPAIR + (int32_t)pair_id) + 1, 1u);
    };
    if (warp == 2) ptx::grid_launch_dependents();      // one warp speaks for the CTA: our own successor may start likewise
    ptx::grid_dependency_wait();                       // C and the split workspace may still be in use by the previous kernel
    const uint32_t quad = warp & 3u;
    const uint32_t ew = warp - 2u;
    const int32_t half = (int32_t)(ew >> 2);
    const uint32_t buf0 = epi0 + ew * EPI_BUFS * kEpiBufBytes;
    const uint32_t tempty0 = PAIR ? ptx::map_to_cta(tempty_bar(0), leader) : tempty_bar(0);
    const bool has_beta_arg = p.beta != 0.f;
    const bool has_acc = nkb > 0;
    const bool scale = p.alpha != 1.f;
    const float alpha = p.alpha, beta = p.beta;
    // where this thread's j-th 16-byte piece of a 128-byte row goes (swizzled); recomputed at every use:
    // eight precomputed addresses would be eight registers held across the whole role
    const uint32_t my_row = buf0 + lane * 128u, my_xor = (lane & 7u) << 4;
    auto piece = [&](int j) { return my_row + (((uint32_t)j << 4) ^ my_xor); };
    // running chunk counter: staging buffer g % EPI_BUFS; bit b of cin_phase = the phase of buffer b's C_in
    // barrier (a tile whose parts are added onto C fetches no C_in, so the phases do not follow g)
    uint32_t g = 0, cin_phase = 0;
    const bool two_bufs = EPI_BUFS == 2;
    // No staging buffers at all: the plan found that this run can store its result straight from
    // registers (beta == 0; C, its leading dimension and N are multiples of 32 bytes), one full 32-byte
    // sector per lane and instruction.  Nothing of the epilogue then passes through shared memory, which
    // all goes to the operand ring.
    const bool direct = EPI_BUFS == 0;
    uint32_t acc = 0, acc_ph = 0;

    // Partial accumulators of the K-slices of a tail tile travel through a private fp32 workspace in a
    // layout where a warp's 16-byte pieces are contiguous (coalesced both ways): [tail tile][slot = slice-1]
    // [cta][warp][accumulator][chunk][unit][piece][lane]; a unit is 32 lanes x 32 columns x 4 bytes.
    constexpr uint32_t kUnitBytes = 8u * 512u;
    auto ws_addr = [&](const WorkItem& w, int32_t slice_m1, int32_t r, int32_t i, int32_t q) {
      const uint64_t idx = ((((uint64_t)w.tail_index * (uint32_t)p.work.slots + (uint32_t)slice_m1) * CLUSTER +
                             slot_rank) * kEpiWarps + ew) * (uint32_t)(MREP * ((NCHUNK + 1) / 2) * UPC) +
                           (uint32_t)((r * ((NCHUNK + 1) / 2) + i) * UPC + q);
      return reinterpret_cast<char*>(p.split_ws) + idx * kUnitBytes + lane * 16u;
    };
    // how many of a tile's column chunks are this warp's, given the tile and the warp's first row
    auto chunks_of = [&](int32_t row0, int32_t col0) {
      int32_t nch = 0;  // chunks of the tile that hold any valid column, if this warp's rows exist
      if (row0 < p.M) {
        nch = (p.N - col0 + CW - 1) / CW;
        if (nch > NCHUNK) nch = NCHUNK;
      }
      const int32_t left = nch - half * kHalfChunks;   // this warp's chunks are consecutive: [half * kHalfChunks, ...)
      return left <= 0 ? 0 : (left > kHalfChunks ? kHalfChunks : left);
    };
    // the i-th chunk of this warp.  The two warps of a lane quadrant take the left and the right half of
    // the tile's columns: a warp then writes 512 consecutive bytes of every row within a short time,
    // which the memory system takes better than every other 128-byte piece (measured on a store-only
    // kernel over a 600 MB matrix: +2 to +4 %).
    auto chunk_of = [&](int32_t i) { return half * kHalfChunks + i; };
    // Bounded wait until every warp of every contributing slice of a tail tile has delivered its
    // partials.  One lane polls, with a pause between polls: this can run beside a main loop, whose
    // copy-issuing warps share the instruction issue slots and the memory pipeline with this warp.
    // the run count of a tail tile's counters, read by lane 0 (see wait_partials); asked for early -- at the
    // top of the owning item, a main loop before the answer is needed -- so that its round trip to L2 is
    // not added to the wait
    auto owner_run_of = [&](const WorkItem& w) {
      uint32_t run = 0;
      if (lane == 0) run = ptx::ld_acquire_gpu(p.split_flags + 2 * (w.tail_index * NPAIR + (int32_t)pair_id) + 1) / kOwnerWarps;
      return run;
    };
    auto wait_partials = [&](const WorkItem& w, int32_t r, uint32_t run) {
      // Two words per tail tile (and pair): arrivals of contributing warps, and owner warps that are done with
      // the tile's partial sums.  Both only grow.  Every warp of the owning CTA group adds one to the second
      // word per run, so its value tells which run of the plan this is without any word from the host: the
      // counters work the same when the launches are replayed from a CUDA graph.  (A warp reads the word
      // before it adds its own one, and at most kOwnerWarps - 1 others have added theirs by then.)
      const uint32_t* flag = p.split_flags + 2 * (w.tail_index * NPAIR + (int32_t)pair_id);
      const uint32_t target = (run + 1u) * p.split_arrivals * (uint32_t)(w.slices - 1);   // lane 0's is the real one
      const long long t_start = clock64();
      uint32_t spins = 0;
      for (;;) {
        bool ready = lane == 0 && (int32_t)(ptx::ld_acquire_gpu(flag) - target) >= 0;
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          (void)ptx::ld_acquire_gpu(flag);  // every lane orders its own reads of the partials after the counter
          return true;
        }
        __nanosleep(200);
        if ((++spins & 63u) == 0u) {
          bool give_up = *(volatile uint32_t*)p.status != kStatusOk;
          if (!give_up && (uint64_t)(clock64() - t_start) > p.timeout_cycles) {
            if (atomicCAS(p.status, (uint32_t)kStatusOk, (uint32_t)kStatusTimeout) == kStatusOk) {
              p.status[1] = kRoleEpiloguePartials;
              p.status[2] = (uint32_t)w.tail_index;
              p.status[3] = (uint32_t)w.tile;
              p.status[4] = (uint32_t)r;
              p.status[5] = blockIdx.x;
              __threadfence();
            }
            give_up = true;
          }
          if (__any_sync(0xffffffffu, give_up)) return false;
        }
      }
    };

    for (int64_t it = 0;; ++it) {
      WorkItem wi;
      EXO_TRACE_TILE(it, 0);
      if (!work_item(p.work, worker, num_workers, it, nkb, &wi)) break;
      EXO_TRACE_TILE(it, 1);
      const int64_t t = wi.tile;
      uint32_t bz;
      const TileCoord tc = tile_coord(t, &bz);
      const int32_t col0 = (tc.n * NPAIR + (int32_t)pair_id) * BN;
      EXO_TRACE_TILE(it, 2);
      if constexpr (MREP == 1) {
        // If this worker's next (and last) item is the owning slice of a tail tile and at least one whole
        // tile came before this one, the other slices' partial sums were published a whole tile's time
        // ago (contributing slices are computed first).  Write their sum into that item's accumulator
        // now, while this item's main loop runs: the MMA warp then accumulates on top of it and the
        // owner's epilogue is an ordinary one.  (With a single whole tile before the slice the partials
        // arrive too late for that; the owner then adds them in its epilogue.)
        WorkItem nx;
        if (it + 1 >= preload_from && !(REDUCE && p.reduce_add) && work_item(p.work, worker, num_workers, it + 1, nkb, &nx) && nx.slices > 1 &&
            nx.slice == 0 && nx.after_whole) {
          uint32_t bz2;
          const TileCoord tc2 = tile_coord(nx.tile, &bz2);
          const int32_t n_mine = chunks_of(tc2.m * (CTA_M * CTA_GROUP) + (int32_t)cta_rank * CTA_M + (int32_t)quad * 32,
                                           (tc2.n * NPAIR + (int32_t)pair_id) * BN);
          if (n_mine > 0) {
            ok = wait_partials(nx, 0, owner_run_of(nx));
            if (!ok) break;
            const uint32_t tnext = tmem_base + ((quad * 32u) << 16) + (acc ^ 1u) * BN;
#pragma unroll 1
            for (int32_t u = 0; u < n_mine * UPC * 2; ++u) {  // 16 columns at a time and rolled: this runs
              // beside a main loop and must not raise the kernel's register count
              const int32_t i = u / (UPC * 2), q = (u / 2) % UPC, h = u & 1;
              uint32_t sum[16];
              for (int32_t sm1 = 0; sm1 < nx.slices - 1; ++sm1) {  // in slice order
                const char* src = ws_addr(nx, sm1, 0, i, q) + h * 2048;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  uint32_t a0, a1, a2, a3;
                  ptx::ld_global_cg_v4(src + j * 512, a0, a1, a2, a3);
                  if (sm1 == 0) {
                    sum[4 * j + 0] = a0; sum[4 * j + 1] = a1; sum[4 * j + 2] = a2; sum[4 * j + 3] = a3;
                  } else {
                    sum[4 * j + 0] = __float_as_uint(__uint_as_float(sum[4 * j + 0]) + __uint_as_float(a0));
                    sum[4 * j + 1] = __float_as_uint(__uint_as_float(sum[4 * j + 1]) + __uint_as_float(a1));
                    sum[4 * j + 2] = __float_as_uint(__uint_as_float(sum[4 * j + 2]) + __uint_as_float(a2));
                    sum[4 * j + 3] = __float_as_uint(__uint_as_float(sum[4 * j + 3]) + __uint_as_float(a3));
                  }
                }
              }
              ptx::tmem_st_32x16(tnext + (uint32_t)(chunk_of(i) * CW + q * 32 + h * 16), sum);
            }
            ptx::tmem_st_wait();
          }
          partials_consumed(nx.tail_index);
          // every epilogue warp of the CTA group reports "filled" to the MMA-issuing CTA
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (ptx::elect_one()) {
            if constexpr (PAIR) ptx::mbar_arrive_cluster(ptx::map_to_cta(tfilled_bar, leader));
            else ptx::mbar_arrive(tfilled_bar);
          }
        }
      }
      EXO_TRACE_TILE(it, 3);
      const bool preloaded = MREP == 1 && wi.slices > 1 && wi.slice == 0 && wi.after_whole && it >= preload_from && !(REDUCE && p.reduce_add);  // see above
      uint32_t owner_run = 0;
      if (wi.slices > 1 && wi.slice == 0 && !preloaded && !(REDUCE && p.reduce_add)) owner_run = owner_run_of(wi);
      // one pass per accumulator of the tile: a single one, or (tall tile) rows 0..127 then 128..255 of the CTA
#pragma unroll 1
      for (int32_t r = 0; r < MREP; ++r) {
      const uint32_t cur = MREP == 1 ? acc : (uint32_t)r;
      const int32_t row0 = tc.m * (CTA_M * CTA_GROUP) + (int32_t)cta_rank * CTA_M + r * kBlockM + (int32_t)quad * 32;
      const int32_t mine = chunks_of(row0, col0);  // how many of the tile's chunks are this warp's
      EXO_TRACE_TILE(it, 4);
      if (has_acc) {
        ok = wait_barrier<PAIR>(tfull_bar(cur), acc_ph, p, WaitSite{kRoleEpilogue, 200 + cur, (uint32_t)t, 0});
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ptx::tc_fence_after_sync();
      }
      if (warp == 2 && lane == 0) EXO_TRACE(2, it, 0, 4096);
      auto release_acc = [&]() {
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (ptx::elect_one()) {
          if constexpr (PAIR) ptx::mbar_arrive_cluster(tempty0 + 8u * cur);
          else ptx::mbar_arrive(tempty0 + 8u * cur);
        }
      };
      const uint32_t tacc = tmem_base + ((quad * 32u) << 16) + cur * BN;
      // unit q of this warp's i-th chunk: 32 accumulator columns
      auto tmem_load = [&](uint32_t (&dst)[32], int32_t i, int32_t q) {  // asynchronous until tmem_ld_wait()
        ptx::tmem_ld_32x32(tacc + (uint32_t)(chunk_of(i) * CW + q * 32), dst);
      };
      if (mine == 0 && has_acc) release_acc();

      // ---- a slice of a tail tile (the tile's K range is cut into wi.slices parts)
      // The unordered alternative (the form of the paper's Section 6 split-K kernels): every part of a cut
      // tile adds alpha * (its partial sum) onto C with a TMA reduce-add; C holds beta * C_in (beta == 1) or
      // zeros (the host cleared it) before the launch, nobody waits for anybody, and the order of the
      // additions, hence the last bits of the result, is left to the memory system.
      const bool tile_reduce = REDUCE && p.reduce_add != 0 && wi.slices > 1;
      const bool has_beta = has_beta_arg && !tile_reduce;
      const bool contributor = wi.slices > 1 && wi.slice != 0 && !tile_reduce;
      const bool owner = wi.slices > 1 && wi.slice == 0 && !preloaded && !tile_reduce;  // has to add the partials itself
      if (contributor) {
        // raw accumulators out, then one arrival per warp on the tile's counter
        for (int32_t i = 0; i < mine; ++i) {
#pragma unroll
          for (int32_t q = 0; q < UPC; ++q) {
            uint32_t raw[32];
            tmem_load(raw, i, q);
            ptx::tmem_ld_wait();
            if (i + 1 == mine && q == UPC - 1) release_acc();
            char* dst = ws_addr(wi, wi.slice - 1, r, i, q);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              ptx::st_global_v4(dst + j * 512, raw[4 * j + 0], raw[4 * j + 1], raw[4 * j + 2], raw[4 * j + 3]);
          }
        }
        __threadfence();  // each lane's partials are visible GPU-wide before the arrival below
        __syncwarp();
        if (ptx::elect_one()) ptx::red_release_gpu_add(p.split_flags + 2 * (wi.tail_index * NPAIR + (int32_t)pair_id), 1u);
        continue;
      }
      if (owner && mine > 0) {
        ok = wait_partials(wi, r, owner_run);
        if (!ok) break;
      }
      auto issue_cin = [&](uint32_t gg, int32_t i) {  // elected lane only: C_in of this warp's i-th chunk
        const uint32_t b = two_bufs ? (gg & 1u) : 0u;
        ptx::mbar_arrive_expect_tx(cin_bar(ew, b), kEpiBufBytes);
        if (batched) ptx::tma_load_3d(buf0 + b * kEpiBufBytes, &tm_c, col0 + chunk_of(i) * CW, row0, (int32_t)bz, cin_bar(ew, b));
        else ptx::tma_load_2d(buf0 + b * kEpiBufBytes, &tm_c, col0 + chunk_of(i) * CW, row0, cin_bar(ew, b));
      };
      if (mine > 0 && has_beta && two_bufs && !direct) {
        if (ptx::elect_one()) {
          ptx::bulk_wait_read<0>();
          issue_cin(g, 0);
        }
      }
      // The chunk loop stays rolled: eight warps interleave, which hides the TMEM load
      // latency as well as a software pipeline did, at a fraction of the code size.
      uint32_t v[UPC][32];
      // An owner that adds the partial sums itself keeps the first contributing slice's next unit on its
      // way from L2 while it converts and stores the current one (one round trip per unit otherwise).
      // Only where a chunk is one unit (fp32 C): with two units in registers the 32 more do not fit into
      // the 168 registers a thread of this kernel can have (352 threads are allocated as 384).
      constexpr bool kPrefetchPartials = UPC == 1;
      uint32_t pf[kPrefetchPartials ? 32 : 1];
      auto prefetch_partial = [&](int32_t i, int32_t q) {
        if constexpr (kPrefetchPartials) {
          const char* src = ws_addr(wi, 0, r, i, q);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            ptx::ld_global_cg_v4(src + j * 512, pf[4 * j + 0], pf[4 * j + 1], pf[4 * j + 2], pf[4 * j + 3]);
        }
      };
      if (owner && mine > 0) prefetch_partial(0, 0);
#pragma unroll 1
      for (int32_t i = 0; i < mine; ++i) {
        if (ok) {
          const int32_t col = col0 + chunk_of(i) * CW;
          const uint32_t b = two_bufs ? (g & 1u) : 0u;
          const uint32_t boff = b * kEpiBufBytes;
          // this thread's row of C (direct stores only)
          char* const c_row = reinterpret_cast<char*>(p.c_ptr) + (int64_t)bz * p.c_batch_bytes +
                              (int64_t)(row0 + (int32_t)lane) * p.ldc_bytes + (int64_t)col * (OUT == kOutFp32 ? 4 : 2);
          const bool row_ok = row0 + (int32_t)lane < p.M;
          // A staging buffer is free once the store that last used it has read it out.
          if (direct) {
          } else if (ptx::elect_one()) {
            if (has_beta) {
              if (two_bufs) {  // prefetch the next chunk's C_in into the other buffer
                if (i + 1 < mine) {
                  ptx::bulk_wait_read<0>();
                  issue_cin(g + 1, i + 1);
                }
              } else {
                ptx::bulk_wait_read<0>();
                issue_cin(g, i);
              }
            } else {
              if (two_bufs) ptx::bulk_wait_read<1>();
              else ptx::bulk_wait_read<0>();
            }
          }
          __syncwarp();
          EXO_TRACE_CHUNK(g, 0);
          if (has_beta && !direct) {
            ok = wait_barrier<false>(cin_bar(ew, b), (cin_phase >> b) & 1u, p,
                                     WaitSite{kRoleEpilogueCin, 300 + b, (uint32_t)t, (uint32_t)i});
            ok = __all_sync(0xffffffffu, ok);
            cin_phase ^= 1u << b;
          }
#pragma unroll
          for (int32_t q = 0; q < UPC; ++q) {
            uint32_t(&cur)[32] = v[q];
            if (has_acc) {
              if (q == 0) {
#pragma unroll
                for (int32_t qq = 0; qq < UPC; ++qq) tmem_load(v[qq], i, qq);
                ptx::tmem_ld_wait();
                EXO_TRACE_CHUNK(g, 1);
                if (i + 1 == mine) release_acc();  // this warp's last read of the accumulator: hand it back early
              }
            } else {
#pragma unroll
              for (int k = 0; k < 32; ++k) cur[k] = 0u;
            }
            if (owner) {  // add the other slices' partial sums, in slice order
              if constexpr (kPrefetchPartials) {
#pragma unroll
                for (int k = 0; k < 32; ++k) cur[k] = __float_as_uint(__uint_as_float(cur[k]) + __uint_as_float(pf[k]));
                if (i + 1 < mine) prefetch_partial(i + 1, 0);
              }
              for (int32_t sm1 = kPrefetchPartials ? 1 : 0; sm1 < wi.slices - 1; ++sm1) {
                const char* src = ws_addr(wi, sm1, r, i, q);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  uint32_t a0, a1, a2, a3;
                  ptx::ld_global_cg_v4(src + j * 512, a0, a1, a2, a3);
                  cur[4 * j + 0] = __float_as_uint(__uint_as_float(cur[4 * j + 0]) + __uint_as_float(a0));
                  cur[4 * j + 1] = __float_as_uint(__uint_as_float(cur[4 * j + 1]) + __uint_as_float(a1));
                  cur[4 * j + 2] = __float_as_uint(__uint_as_float(cur[4 * j + 2]) + __uint_as_float(a2));
                  cur[4 * j + 3] = __float_as_uint(__uint_as_float(cur[4 * j + 3]) + __uint_as_float(a3));
                }
              }
            }
            if (scale) {
#pragma unroll
              for (int k = 0; k < 32; ++k) cur[k] = __float_as_uint(alpha * __uint_as_float(cur[k]));
            }
            if (ok && direct) {
              // 32 accumulator columns of this thread's row: 128 bytes (fp32) or 64 bytes (16-bit) of C, as
              // 32-byte pieces.  N is a multiple of a piece, so a piece lies inside the matrix or outside.
              if constexpr (OUT == kOutFp32) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  if (row_ok && col + q * 32 + 8 * j < p.N) ptx::st_global_v8(c_row + q * 128 + j * 32, &cur[8 * j]);
              } else {
                uint32_t w[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k] = pack2<OUT>(__uint_as_float(cur[2 * k]), __uint_as_float(cur[2 * k + 1]));
#pragma unroll
                for (int j = 0; j < 2; ++j)
                  if (row_ok && col + q * 32 + 16 * j < p.N) ptx::st_global_v8(c_row + q * 64 + j * 32, &w[8 * j]);
              }
            } else if (ok) {
              if constexpr (OUT == kOutFp32) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  if (has_beta) {
                    uint32_t c0, c1, c2, c3;
                    ptx::ld_shared_v4(piece(j) + boff, c0, c1, c2, c3);
                    cur[4 * j + 0] = __float_as_uint(fmaf(beta, __uint_as_float(c0), __uint_as_float(cur[4 * j + 0])));
                    cur[4 * j + 1] = __float_as_uint(fmaf(beta, __uint_as_float(c1), __uint_as_float(cur[4 * j + 1])));
                    cur[4 * j + 2] = __float_as_uint(fmaf(beta, __uint_as_float(c2), __uint_as_float(cur[4 * j + 2])));
                    cur[4 * j + 3] = __float_as_uint(fmaf(beta, __uint_as_float(c3), __uint_as_float(cur[4 * j + 3])));
                  }
                  ptx::st_shared_v4(piece(j) + boff, cur[4 * j + 0], cur[4 * j + 1], cur[4 * j + 2], cur[4 * j + 3]);
                }
              } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {  // 32 columns = four 16-byte pieces of 8 halves
                  const uint32_t addr = piece(4 * q + j) + boff;
                  float x[8];
#pragma unroll
                  for (int k = 0; k < 8; ++k) x[k] = __uint_as_float(cur[8 * j + k]);
                  if (has_beta) {
                    uint32_t cw[4];
                    ptx::ld_shared_v4(addr, cw[0], cw[1], cw[2], cw[3]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                      const float2 cc = unpack2<OUT>(cw[k]);
                      x[2 * k] = fmaf(beta, cc.x, x[2 * k]);
                      x[2 * k + 1] = fmaf(beta, cc.y, x[2 * k + 1]);
                    }
                  }
                  ptx::st_shared_v4(addr, pack2<OUT>(x[0], x[1]), pack2<OUT>(x[2], x[3]), pack2<OUT>(x[4], x[5]),
                                    pack2<OUT>(x[6], x[7]));
                }
              }
            }
          }
          EXO_TRACE_CHUNK(g, 2);
          if (ok && !direct) {
            ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the TMA store
            __syncwarp();
            if (ptx::elect_one()) {
              if (tile_reduce) {
                if (batched) ptx::tma_reduce_add_3d(&tm_c, col, row0, (int32_t)bz, buf0 + boff);
                else ptx::tma_reduce_add_2d(&tm_c, col, row0, buf0 + boff);
              } else if (p.c_evict_first) {
                if (batched) ptx::tma_store_3d_hint(&tm_c, col, row0, (int32_t)bz, buf0 + boff, ptx::policy_evict_first());
                else ptx::tma_store_2d_hint(&tm_c, col, row0, buf0 + boff, ptx::policy_evict_first());
              } else if (batched) {
                ptx::tma_store_3d(&tm_c, col, row0, (int32_t)bz, buf0 + boff);
              } else {
                ptx::tma_store_2d(&tm_c, col, row0, buf0 + boff);
              }
              ptx::bulk_commit();
            }
            EXO_TRACE_CHUNK(g, 3);
            ++g;
          }
          if (direct) { EXO_TRACE_CHUNK(g, 3); ++g; }
          (void)c_row; (void)row_ok;
        }
      }
      if (!ok) break;
      }  // accumulators of the tile
      if (!ok) break;
      if (wi.slices > 1 && wi.slice == 0 && !preloaded && !(REDUCE && p.reduce_add)) partials_consumed(wi.tail_index);
      if (warp == 2 && lane == 0) EXO_TRACE(2, it, 1, 4096);
      if (MREP == 2 || (acc ^= 1u) == 0u) acc_ph ^= 1u;
    }
    __syncwarp();
    // The stores must have read their staging buffers before this CTA's shared memory goes away;
    // their global writes complete on their own and are visible when the kernel has ended.
    if (ptx::elect_one()) ptx::bulk_wait_read<0>();
    __syncwarp();
  }

  // ---------------------------------------------------------------- teardown
  if (!ok) {
    // This thread abandoned a wait: give copies and MMAs still in flight time to land before shared
    // and tensor memory are released.  (Every thread that gives up passes here with ok == false, and
    // the barriers below hold the rest of the CTA and of the cluster back until it has slept; reading
    // the status word from global memory instead would put a memory round trip on every CTA's exit.)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if constexpr (PAIR) {  // the peer's shared and tensor memory stay valid until both CTAs are done
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<CTA_GROUP>(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0) EXO_TRACE(2, 4095, 1, 4096);
}

}  // namespace exo
