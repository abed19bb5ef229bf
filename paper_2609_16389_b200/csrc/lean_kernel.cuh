// One-tile-per-CTA tcgen05 GEMM kernel for problems of less than one wave (sm_100a).
//
// The persistent kernel of gemm_kernel.cuh is built for throughput: on a problem of a few dozen
// tiles and a short K loop its run time is a chain of latencies (set-up, first copy, first data,
// last MMA, drain, exit), and the paper's Section 6 singles out exactly these small matrices as the
// regime where kernels differ most.  This kernel computes one 128 x BN tile per CTA and shortens
// every link of that chain:
//
//   warp 0             initialises the barriers and issues the copies of the first two k-blocks BEFORE
//                      the CTA-wide set-up barrier (nothing but this warp's own barriers is needed for
//                      that), then the remaining k-blocks, waiting only for stages that are reused
//   warp 1             allocates tensor memory, issues the MMAs (one elected lane), frees tensor
//                      memory as soon as every epilogue warp has read its part of the accumulator
//   warps 2..          epilogue, four or eight warps: C_in (beta != 0) is fetched while the main loop
//                      runs, every warp has a staging buffer per column chunk of its own (no buffer
//                      is ever waited for), and a warp leaves as soon as its own store has read its
//                      buffer: without a cluster there is no barrier at the end
//
// K split across a cluster (the cluster's size, 1, 2 or 4, is the split factor): the CTAs of a cluster
// compute the same tile over consecutive ranges of k-blocks, each into its own TMEM accumulator, and
// reduce-scatter the partial sums by rows through distributed shared memory: the CTA of rank r
// finishes the rows of TMEM lane quadrant(s) r; every other CTA's warps of that quadrant stage their
// fp32 partials in their own operand ring (free by then) and send them with one bulk copy each
// (cp.async.bulk shared::cta -> shared::cluster, counted in bytes on the receiver's barrier), and the
// finishing CTA adds them in rank order -- deterministic, no global-memory round trip.  (Ordinary
// remote stores were measured first: 20 bytes per clock and SM, 4.5 k clocks for the exchange.)
// A k-block of eight 128 x 64 x 16 MMAs costs the issuing thread about 600 clocks whatever the tensor
// core could do, so a short problem on few SMs is bound by the number of MMAs per CTA; cutting K over
// four SMs cuts that by four for an exchange of 24 KB per CTA.
//
// The code is short on purpose (a CTA runs every basic block exactly once, from a cold instruction
// cache).  Operand staging, descriptors, tensor maps and the parameter block are those of the
// 1-CTA tiles of the persistent kernel; the plan decides which of the two kernels runs.
#pragma once
#include "gemm_kernel.cuh"

namespace exo {

#ifdef EXO_GEMM_TRACE
// stamp k (0..7) of an epilogue warp's lane 0 (CTA 0 only)
#define EXO_TRACE_W(k) do { if (lane == 0) EXO_TRACE(0, 3100 + warp * 8 + (k), 0, 4096); } while (0)
#define EXO_TRACE_M(j, k) do { if (lane == 0) EXO_TRACE(0, 2100 + (j) * 8 + (k), 0, 3000); } while (0)
#else
#define EXO_TRACE_M(j, k) do {} while (0)
#define EXO_TRACE_W(k) do {} while (0)
#endif

template <int BN, int OUT, int KSUB>
__global__ void __launch_bounds__(lean_threads(BN, OUT == kOutFp32 ? 4 : 2), 1)
exo_gemm_lean_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
  static_assert(BN == 64 || BN == 128, "tile N");
  constexpr int C_BYTES = OUT == kOutFp32 ? 4 : 2;
  constexpr int CW = 128 / C_BYTES;                  // columns per chunk = 128 bytes of C
  constexpr int NCHUNK = BN / CW;
  constexpr int EW = lean_epi_warps(BN, C_BYTES);    // epilogue warps
  constexpr int CPW = NCHUNK * 4 / EW;               // chunks per warp: 1 or 2
  constexpr int UPC = CW / 32;                       // 32-column TMEM loads per chunk
  constexpr int STAGE_BYTES = stage_bytes(1, BN, KSUB);
  constexpr int A_BYTES = KSUB * kATileBytes;
  // (One accumulator.  Two, taken in turn by consecutive MMAs and added in the epilogue, were measured: the
  // k-block period stayed at 930 clocks, so the MMAs into one accumulator do not wait for one another.)
  constexpr uint32_t TMEM_COLS = BN;
  constexpr int UNITS = BN / 32;                     // 4 KB units (32 rows x 32 fp32 columns) of a quadrant's partial sums
  const int32_t STAGE_K = (int32_t)p.sub_k * KSUB;
  const int32_t STAGES = p.stages;
  // the CTAs of a cluster share one tile: rank r takes the k-blocks [kb_begin, kb_end)
  const uint32_t S = ptx::cluster_nctarank();        // 1, 2 or 4
  const uint32_t rank = S > 1 ? ptx::cluster_ctarank() : 0u;
  const uint32_t QPC = 4u / S;                       // TMEM lane quadrants whose rows this CTA finishes
  const uint32_t log2_s = S >> 1;                    // S is a power of two
  const int32_t kb_begin = (int32_t)(((int64_t)p.num_k_blocks * rank) >> log2_s);
  const int32_t kb_end = (int32_t)(((int64_t)p.num_k_blocks * (rank + 1u)) >> log2_s);
  const int32_t nkb = kb_end - kb_begin;             // this CTA's k-blocks

  extern __shared__ uint8_t smem_raw[];
  const uint32_t stage0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi0 = stage0 + (uint32_t)STAGES * STAGE_BYTES;
  const uint32_t recv0 = epi0 + 4u * NCHUNK * kEpiBufBytes;   // [source slot][own quadrant][unit] partial sums of the peers
  const uint32_t bar0 = recv0 + (S - 1u) * QPC * UNITS * kEpiBufBytes;
  auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (kMaxStages + s); };
  const uint32_t tfull_bar = bar0 + 8u * (2 * kMaxStages);
  const uint32_t tdone_bar = tfull_bar + 8u;        // every epilogue warp has read its part of the accumulator
  const uint32_t recv_bar = tdone_bar + 8u;         // the peers' partial sums of this CTA's rows have landed
  auto cin_bar = [&](uint32_t w) { return recv_bar + 8u + 8u * w; };
  constexpr uint32_t kBarriers = 2 * kMaxStages + 3 + EW;
  const uint32_t tmem_slot = bar0 + 8u * kBarriers;
  static_assert(8 * kBarriers + 4 <= kBarrierBytes, "barrier area");

  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = threadIdx.x & 31u;
  const TileCoord tc = raster_decode(p.raster, (int64_t)(blockIdx.x >> log2_s));
  const int32_t tile_row0 = tc.m * kBlockM, col0 = tc.n * BN;
  bool ok = true;
  // k-blocks whose copies are issued before the CTA's set-up barrier (two: the copy unit queues about eight
  // boxes; issuing more there would only hold the barrier back)
  const int32_t early = nkb < 2 ? nkb : (STAGES < 2 ? STAGES : 2);
  if (threadIdx.x == 0) EXO_TRACE(2, 4095, 0, 4096);

  // the copies of k-block kb into its stage (elected lane of warp 0 only)
  auto issue_loads = [&](int32_t j, uint32_t s) {   // j-th k-block of this CTA into stage s
    const int32_t kb = kb_begin + j;
    const uint32_t bar = full_bar(s);
    ptx::mbar_arrive_expect_tx(bar, STAGE_BYTES);
    if (p.debug_skip_k_block == kb && blockIdx.x == 0) return;   // test hook: a stage that never fills
    const uint32_t a_dst = stage0 + s * STAGE_BYTES, b_dst = a_dst + A_BYTES;
    const int32_t k0 = kb * STAGE_K;
    constexpr uint32_t MN_BOX_BYTES = KSUB * 8192u;   // M/N-contiguous 16-bit operand: one box of 64 rows
    if (!p.a.mn_major) {
#pragma unroll
      for (int h = 0; h < KSUB; ++h) ptx::tma_load_2d(a_dst + h * kATileBytes, &tm_a, k0 + h * (int32_t)p.sub_k, tile_row0, bar);
    } else if (!p.tf32) {
#pragma unroll
      for (int b = 0; b < 2; ++b) ptx::tma_load_2d(a_dst + b * MN_BOX_BYTES, &tm_a, tile_row0 + 64 * b, k0, bar);
    } else {
#pragma unroll
      for (int b = 0; b < 4; ++b) ptx::tma_load_2d(a_dst + b * (MN_BOX_BYTES / 2), &tm_a, tile_row0 + 32 * b, k0, bar);
    }
    if (!p.b.mn_major) {
#pragma unroll
      for (int h = 0; h < KSUB; ++h) ptx::tma_load_2d(b_dst + h * (BN * 128), &tm_b, k0 + h * (int32_t)p.sub_k, col0, bar);
    } else if (!p.tf32) {
#pragma unroll
      for (int b = 0; b < BN / 64; ++b) ptx::tma_load_2d(b_dst + b * MN_BOX_BYTES, &tm_b, col0 + 64 * b, k0, bar);
    } else {
#pragma unroll
      for (int b = 0; b < BN / 32; ++b) ptx::tma_load_2d(b_dst + b * (MN_BOX_BYTES / 2), &tm_b, col0 + 32 * b, k0, bar);
    }
  };

  // ---------------------------------------------------------------- set-up
  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tm_a);
      ptx::prefetch_tensormap(&tm_b);
      ptx::grid_launch_dependents();   // the next kernel's own set-up may overlap this whole kernel
    }
    for (uint32_t i = lane; i < kBarriers; i += 32u) {
      uint32_t count = 1u;
      if (i == 2 * kMaxStages + 1) count = (uint32_t)EW;                             // tdone: every epilogue warp
      ptx::mbar_init(bar0 + 8u * i, count);
    }
    ptx::fence_mbar_init();
    // recv: one arrival (here) plus the bytes of the peers' partial sums of this CTA's quadrants
    if (S > 1 && lane == 0) ptx::mbar_arrive_expect_tx(recv_bar, (S - 1u) * QPC * UNITS * kEpiBufBytes);
    ptx::fence_proxy_async_smem();     // the copies below signal these barriers through the async proxy
    __syncwarp();
    // The operands may be the previous kernel's output; nothing before this line reads global memory.
    ptx::grid_dependency_wait();
    if (ptx::elect_one()) {
      for (int32_t j = 0; j < early; ++j) {
        EXO_TRACE(0, j, 0, 2048);
        issue_loads(j, (uint32_t)j);
        EXO_TRACE(0, j, 1, 2048);
      }
    }
  } else if (warp == 1) {
    ptx::tmem_alloc<1>(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish<1>();
  } else if (warp == 2 && lane == 0) {
    ptx::prefetch_tensormap(&tm_c);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (S > 1) ptx::cluster_arrive();   // this CTA's barriers exist; waited for before the first remote access
  ptx::tc_fence_after_sync();
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot) : "memory");
  // Warp 0 passed the dependency wait before the barrier above, so the kernel in front has ended; the
  // other warps execute the wait themselves (it returns at once) so that each thread's own reads of
  // global memory -- the status word of the bounded waits included -- are ordered after it.
  if (warp != 0) ptx::grid_dependency_wait();
  if (threadIdx.x == 64) EXO_TRACE(2, 4094, 0, 4096);

  if (warp == 0) {
    // ============================================================ producer: k-blocks beyond the first ring
    // (stage and phase as counters: a division by the run-time ring depth costs more than issuing a copy)
    uint32_t s = (uint32_t)early, ph = 0;
    if (s == (uint32_t)STAGES) { s = 0; ph = 1u; }
    for (int32_t j = early; j < nkb && ok; ++j) {
      if (j >= STAGES) {
        ok = wait_barrier<false>(empty_bar(s), ph ^ 1u, p, WaitSite{kRoleProducer, s, blockIdx.x, (uint32_t)(kb_begin + j)});
        ok = __all_sync(0xffffffffu, ok);
      }
      if (ok && ptx::elect_one()) {
        EXO_TRACE(0, j, 0, 2048);
        issue_loads(j, s);
        EXO_TRACE(0, j, 1, 2048);
      }
      if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1u; }
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer and owner of tensor memory
    const uint32_t a_step = p.a.k_step_enc, b_step = p.b.k_step_enc, a_sub = p.a.k_sub_enc, b_sub = p.b.k_sub_enc;
    const bool tf32 = p.tf32 != 0;
    const int32_t umma_k = (int32_t)p.umma_k;
    const uint32_t idesc = p.idesc;
    constexpr int kMmaPerStage = 4 * KSUB;   // an MMA consumes 32 bytes of K whatever the element size
    auto k_off = [](int32_t k, uint32_t step, uint32_t sub) {  // descriptor offset of the k-th MMA of a stage
      return (uint64_t)((uint32_t)(k & 3) * step + (uint32_t)(k >> 2) * sub);
    };
    uint32_t s = 0, ph = 0;
    for (int32_t j = 0; j < nkb && ok; ++j) {
      EXO_TRACE_M(j, 0);
      ok = wait_barrier<false>(full_bar(s), ph, p, WaitSite{kRoleMma, s, blockIdx.x, (uint32_t)(kb_begin + j)});
      EXO_TRACE_M(j, 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      EXO_TRACE_M(j, 2);
      if (ptx::elect_one()) {
        EXO_TRACE(1, j, 0, 2048);
        const uint32_t a_addr = stage0 + s * STAGE_BYTES;
        const uint64_t a_desc = make_smem_desc(a_addr, p.a), b_desc = make_smem_desc(a_addr + A_BYTES, p.b);
        const int32_t k_left = p.K - (kb_begin + j) * STAGE_K;
        if (k_left >= STAGE_K && !tf32) {
#pragma unroll
          for (int32_t k = 0; k < kMmaPerStage; ++k)
            ptx::umma_f16<1>(tmem_base, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc,
                             (j != 0 || k != 0) ? 1u : 0u);
        } else {  // tf32, or a ragged last k-block, which skips the MMAs that would only read zero fill
          const int32_t n_mma = k_left >= STAGE_K ? kMmaPerStage : (k_left + umma_k - 1) / umma_k;
          for (int32_t k = 0; k < n_mma; ++k) {
            const uint32_t accumulate = (j != 0 || k != 0) ? 1u : 0u, d = tmem_base;
            if (tf32) ptx::umma_tf32<1>(d, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc, accumulate);
            else ptx::umma_f16<1>(d, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc, accumulate);
          }
        }
        EXO_TRACE_M(j, 3);
        if (j + STAGES < nkb) ptx::umma_commit<1>(empty_bar(s), 1);   // only a stage that is filled again is released
        if (j == nkb - 1) ptx::umma_commit<1>(tfull_bar, 1);           // accumulator complete
        EXO_TRACE(1, j, 1, 2048);
      }
      __syncwarp();
      if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1u; }
    }
    // Tensor memory goes back as soon as the epilogue warps have read it (they arrive also when they give up).
    const bool drained = wait_barrier<false>(tdone_bar, 0u, p, WaitSite{kRoleMma, 120, blockIdx.x, 0});
    if (!__all_sync(0xffffffffu, drained && ok))
      for (int i = 0; i < 200; ++i) __nanosleep(1000);   // a wait was abandoned: let MMAs in flight land first
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<1>(tmem_base, TMEM_COLS);
    if (lane == 0) EXO_TRACE(0, 3000, 0, 4096);
    ok = true;   // (the pause after an abandoned wait has been taken above)
  } else {
    // ============================================================ epilogue
    const uint32_t ew = warp - 2u;
    const uint32_t quad = warp & 3u;                 // the TMEM lanes a warp may read: 32 * (warp % 4) ..
    const int32_t first_chunk = (int32_t)(ew >> 2) * CPW;
    const int32_t row0 = tile_row0 + (int32_t)quad * 32;
    int32_t mine = 0;                                 // this warp's chunks that hold any valid element
    if (row0 < p.M) {
      const int32_t nch = (p.N - col0 + CW - 1) / CW - first_chunk;
      mine = nch < 0 ? 0 : (nch > CPW ? CPW : nch);
    }
    const uint32_t buf0 = epi0 + (quad * NCHUNK + (uint32_t)first_chunk) * kEpiBufBytes;
    const bool has_beta = p.beta != 0.f, has_acc = nkb > 0, scale = p.alpha != 1.f;
    const float alpha = p.alpha, beta = p.beta;
    const uint32_t owner = quad / QPC;               // the rank that finishes this warp's rows
    const bool finish = owner == rank;
    EXO_TRACE_W(0);
    if (S > 1) ptx::cluster_wait();                  // every CTA of the cluster has initialised its barriers
    EXO_TRACE_W(1);
    if (has_beta && finish && mine > 0 && ptx::elect_one()) {   // C_in of all of this warp's chunks, while the main loop runs
      ptx::mbar_arrive_expect_tx(cin_bar(ew), (uint32_t)mine * kEpiBufBytes);
      for (int32_t i = 0; i < mine; ++i)
        ptx::tma_load_2d(buf0 + (uint32_t)i * kEpiBufBytes, &tm_c, col0 + (first_chunk + i) * CW, row0, cin_bar(ew));
    }
    __syncwarp();
    if (has_acc) {
      ok = wait_barrier<false>(tfull_bar, 0u, p, WaitSite{kRoleEpilogue, 200, blockIdx.x, 0});
      ok = __all_sync(0xffffffffu, ok);
      ptx::tc_fence_after_sync();
    }
    if (warp == 2 && lane == 0) EXO_TRACE(2, 0, 0, 4096);
    EXO_TRACE_CHUNK(0, 0);
    uint32_t v[CPW][UPC][32];
    if (ok && has_acc && (mine > 0 || S > 1)) {   // (a cluster exchanges all of a quadrant's columns, valid or not)
      const uint32_t tacc = tmem_base + ((quad * 32u) << 16);
#pragma unroll
      for (int i = 0; i < CPW; ++i)
#pragma unroll
        for (int q = 0; q < UPC; ++q)
          if (i < mine || S > 1) ptx::tmem_ld_32x32(tacc + (uint32_t)((first_chunk + i) * CW + q * 32), v[i][q]);
      ptx::tmem_ld_wait();
    } else {
#pragma unroll
      for (int i = 0; i < CPW; ++i)
#pragma unroll
        for (int q = 0; q < UPC; ++q)
#pragma unroll
          for (int k = 0; k < 32; ++k) v[i][q][k] = 0u;
    }
    EXO_TRACE_CHUNK(0, 1);
    EXO_TRACE_W(2);
    const uint32_t my_xor = (lane & 7u) << 4;
    if (S > 1) {
      // partial sums travel as 4 KB units (32 rows x 32 fp32 columns): lane l's 128 bytes at l * 128, 16-byte pieces swizzled
      const uint32_t my_piece0 = lane * 128u;
      const uint32_t first_unit = (uint32_t)first_chunk * UPC;
      if (!finish) {
        // Hand this warp's partial sums to the CTA that finishes these rows: staged in this CTA's own operand
        // ring (its MMAs have completed, so the ring is free), then one bulk copy into the peer's receive buffer.
        if (ok) {
          const uint32_t slot = rank < owner ? rank : rank - 1u;
          const uint32_t src = stage0 + (quad * UNITS + first_unit) * kEpiBufBytes;
#pragma unroll
          for (int i = 0; i < CPW; ++i)
#pragma unroll
            for (int q = 0; q < UPC; ++q)
#pragma unroll
              for (int j = 0; j < 8; ++j)
                ptx::st_shared_v4(src + (uint32_t)(i * UPC + q) * kEpiBufBytes + my_piece0 + (((uint32_t)j << 4) ^ my_xor),
                                  v[i][q][4 * j + 0], v[i][q][4 * j + 1], v[i][q][4 * j + 2], v[i][q][4 * j + 3]);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          EXO_TRACE_W(3);
          if (ptx::elect_one())
            ptx::bulk_copy_to_cluster(ptx::map_to_cta(recv0 + ((slot * QPC + (quad % QPC)) * UNITS + first_unit) * kEpiBufBytes, owner), src,
                                      (uint32_t)(CPW * UPC) * kEpiBufBytes, ptx::map_to_cta(recv_bar, owner));
          EXO_TRACE_W(4);
        }
        mine = 0;   // nothing to store
      } else if (ok) {
        EXO_TRACE_W(3);
        ok = wait_barrier<false>(recv_bar, 0u, p, WaitSite{kRoleEpiloguePartials, 400, blockIdx.x, rank});
        ok = __all_sync(0xffffffffu, ok);
        EXO_TRACE_W(4);
        if (ok) {
#pragma unroll 1
          for (uint32_t slot = 0; slot + 1u < S; ++slot) {   // in rank order
            const uint32_t src = recv0 + ((slot * QPC + (quad % QPC)) * UNITS + first_unit) * kEpiBufBytes + my_piece0;
#pragma unroll
            for (int i = 0; i < CPW; ++i)
#pragma unroll
              for (int q = 0; q < UPC; ++q)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  uint32_t a0, a1, a2, a3;
                  ptx::ld_shared_v4(src + (uint32_t)(i * UPC + q) * kEpiBufBytes + (((uint32_t)j << 4) ^ my_xor), a0, a1, a2, a3);
                  v[i][q][4 * j + 0] = __float_as_uint(__uint_as_float(v[i][q][4 * j + 0]) + __uint_as_float(a0));
                  v[i][q][4 * j + 1] = __float_as_uint(__uint_as_float(v[i][q][4 * j + 1]) + __uint_as_float(a1));
                  v[i][q][4 * j + 2] = __float_as_uint(__uint_as_float(v[i][q][4 * j + 2]) + __uint_as_float(a2));
                  v[i][q][4 * j + 3] = __float_as_uint(__uint_as_float(v[i][q][4 * j + 3]) + __uint_as_float(a3));
                }
          }
        }
      }
    }
    EXO_TRACE_W(5);
    if (ok && has_beta && mine > 0) {
      ok = wait_barrier<false>(cin_bar(ew), 0u, p, WaitSite{kRoleEpilogueCin, 300, blockIdx.x, 0});
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
#pragma unroll
      for (int i = 0; i < CPW; ++i) {
        if (i < mine) {
          const uint32_t my_row = buf0 + (uint32_t)i * kEpiBufBytes + lane * 128u;
          auto piece = [&](int j) { return my_row + (((uint32_t)j << 4) ^ my_xor); };   // 128-byte swizzle
#pragma unroll
          for (int q = 0; q < UPC; ++q) {
            uint32_t(&cur)[32] = v[i][q];
            if (scale) {
#pragma unroll
              for (int k = 0; k < 32; ++k) cur[k] = __float_as_uint(alpha * __uint_as_float(cur[k]));
            }
            if constexpr (OUT == kOutFp32) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                if (has_beta) {
                  uint32_t c0, c1, c2, c3;
                  ptx::ld_shared_v4(piece(j), c0, c1, c2, c3);
                  cur[4 * j + 0] = __float_as_uint(fmaf(beta, __uint_as_float(c0), __uint_as_float(cur[4 * j + 0])));
                  cur[4 * j + 1] = __float_as_uint(fmaf(beta, __uint_as_float(c1), __uint_as_float(cur[4 * j + 1])));
                  cur[4 * j + 2] = __float_as_uint(fmaf(beta, __uint_as_float(c2), __uint_as_float(cur[4 * j + 2])));
                  cur[4 * j + 3] = __float_as_uint(fmaf(beta, __uint_as_float(c3), __uint_as_float(cur[4 * j + 3])));
                }
                ptx::st_shared_v4(piece(j), cur[4 * j + 0], cur[4 * j + 1], cur[4 * j + 2], cur[4 * j + 3]);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 4; ++j) {   // 32 columns = four 16-byte pieces of 8 halves
                const uint32_t addr = piece(4 * q + j);
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
          EXO_TRACE_CHUNK(i, 2);
          ptx::fence_proxy_async_smem();   // generic-proxy writes -> visible to the TMA store
          __syncwarp();
          if (ptx::elect_one()) {
            ptx::tma_store_2d(&tm_c, col0 + (first_chunk + i) * CW, row0, buf0 + (uint32_t)i * kEpiBufBytes);
            ptx::bulk_commit();
          }
          EXO_TRACE_CHUNK(i, 3);
        }
      }
    }
    // This warp has read its part of the accumulator (long ago: the arrival is kept off the path to the
    // stores; tensor memory is only wanted back at the CTA's exit).  Also on the way out of an abandoned wait.
    ptx::tc_fence_before_sync();
    __syncwarp();
    if (ptx::elect_one()) ptx::mbar_arrive(tdone_bar);
    if (ok) {
      // the stores must have read this warp's buffers before the warp (possibly the CTA's last) leaves
      if (warp == 2 && lane == 0) EXO_TRACE(2, 0, 1, 4096);
      if (ptx::elect_one()) ptx::bulk_wait_read<0>();
      __syncwarp();
      if (warp == 2 && lane == 0) EXO_TRACE(2, 4095, 1, 4096);
    }
  }
  // A thread that gave up a wait lets copies still in flight land before it leaves: shared memory stays
  // until the CTA's last thread has gone.
  if (!ok)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  if (S > 1) {
    // No CTA leaves while a peer may still write into its receive buffer or arrive on its barrier.
    // (Warps 0 and 1 have not yet waited for the set-up phase of the cluster barrier.)
    if (warp < 2) ptx::cluster_wait();
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
}

}  // namespace exo
