// One-tile-per-CTA-pair tcgen05 GEMM kernel for problems of at most one wave of 2-CTA tiles (sm_100a).
//
// The form of lean_kernel.cuh for tiles of 256 x BN computed by a pair of CTAs on two SMs (tcgen05
// cta_group::2: each CTA stages its own 128 rows of A and its own half of B, the leader's thread issues
// the MMAs of both).  A one-wave problem runs the persistent kernel's set-up, scheduler and two-accumulator
// hand-over for nothing, and its run is a chain of latencies (the paper's Section 6 points at such shapes as
// the ones where kernels differ most): first MMA 3.6 k clocks after the start, the epilogue 750 clocks after
// the accumulator is complete, the exit 2.1 k clocks after the last store is issued.  Here
//
//   warp 0             initialises the barriers; in the leading CTA it issues the copies of the first two
//                      k-blocks BEFORE any barrier (its copies signal its own barriers), in the other CTA
//                      right after the cluster's set-up barrier; then the remaining k-blocks
//   warp 1             allocates tensor memory; in the leading CTA issues the MMAs; frees tensor memory
//   warps 2..9         epilogue: once the accumulator is complete the operand ring is idle, so every chunk of
//                      every warp is staged in a buffer of its own there: no store is waited for, C_in
//                      (beta != 0) of all of a warp's chunks is fetched at once
//
// One accumulator, no scheduler, no K split.  Operand staging, descriptors, tensor maps and the parameter
// block are those of the persistent kernel's 2-CTA tiles; the plan decides which kernel runs.
#pragma once
#include "gemm_kernel.cuh"

namespace exo {

template <int BN, int OUT, int KSUB>
__global__ void __launch_bounds__(kLeanPairThreads, 1)
exo_gemm_lean_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                          const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
  static_assert(BN == 128 || BN == 256, "tile N");
  constexpr int C_BYTES = OUT == kOutFp32 ? 4 : 2;
  constexpr int CW = 128 / C_BYTES;                  // columns per chunk = 128 bytes of C
  constexpr int NCHUNK = BN / CW;                    // 2, 4 or 8
  constexpr int EW = 8;                              // epilogue warps: two per TMEM lane quadrant
  constexpr int CPW = NCHUNK / 2;                    // chunks per warp: 1, 2 or 4
  constexpr int UPC = CW / 32;                       // 32-column TMEM loads per chunk
  constexpr int B_ROWS = BN / 2;                     // rows of the B tile this CTA stages
  constexpr int STAGE_BYTES = stage_bytes(2, BN, KSUB);
  constexpr int A_BYTES = KSUB * kATileBytes;
  constexpr uint32_t TMEM_COLS = BN;
  const int32_t STAGE_K = (int32_t)p.sub_k * KSUB;
  const int32_t STAGES = p.stages;
  const int32_t nkb = p.num_k_blocks;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t stage0 = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = stage0 + (uint32_t)lean_pair_ring_bytes(BN, KSUB, STAGES, C_BYTES);
  auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (kMaxStages + s); };
  const uint32_t tfull_bar = bar0 + 8u * (2 * kMaxStages);
  const uint32_t tdone_bar = tfull_bar + 8u;        // every epilogue warp of this CTA has read its part of the accumulator
  auto cin_bar = [&](uint32_t w) { return tdone_bar + 8u + 8u * w; };
  constexpr uint32_t kBarriers = 2 * kMaxStages + 2 + EW;
  const uint32_t tmem_slot = bar0 + 8u * kBarriers;
  static_assert(8 * kBarriers + 4 <= kBarrierBytes, "barrier area");

  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t cta_rank = ptx::cluster_ctarank();  // 0: the CTA whose thread issues the MMAs
  const TileCoord tc = raster_decode(p.raster, (int64_t)(blockIdx.x >> 1));
  const int32_t cta_row0 = tc.m * (2 * kBlockM) + (int32_t)cta_rank * kBlockM, col0 = tc.n * BN;
  const int32_t b_row0 = col0 + (int32_t)cta_rank * B_ROWS;
  const uint32_t leader_full0 = ptx::map_to_cta(full_bar(0), 0u);   // both CTAs' copies count on the leader's barriers
  bool ok = true;
  const int32_t early = nkb < 2 ? nkb : (STAGES < 2 ? STAGES : 2);  // k-blocks copied ahead of the main loop's start
  if (threadIdx.x == 0) EXO_TRACE(2, 4095, 0, 4096);

  // the copies of k-block kb into stage s (elected lane of warp 0 only)
  auto issue_loads = [&](int32_t kb, uint32_t s) {
    if (cta_rank == 0) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);
    if (p.debug_skip_k_block == kb && blockIdx.x == 0) return;   // test hook: a stage that never fills
    const uint32_t a_dst = stage0 + s * STAGE_BYTES, b_dst = a_dst + A_BYTES, bar = leader_full0 + 8u * s;
    const int32_t k0 = kb * STAGE_K;
    constexpr uint32_t MN_BOX_BYTES = KSUB * 8192u;   // M/N-contiguous 16-bit operand: one box of 64 rows
    if (!p.a.mn_major) {
#pragma unroll
      for (int h = 0; h < KSUB; ++h) ptx::tma_load_2d_pair(a_dst + h * kATileBytes, &tm_a, k0 + h * (int32_t)p.sub_k, cta_row0, bar);
    } else if (!p.tf32) {
#pragma unroll
      for (int b = 0; b < 2; ++b) ptx::tma_load_2d_pair(a_dst + b * MN_BOX_BYTES, &tm_a, cta_row0 + 64 * b, k0, bar);
    } else {
#pragma unroll
      for (int b = 0; b < 4; ++b) ptx::tma_load_2d_pair(a_dst + b * (MN_BOX_BYTES / 2), &tm_a, cta_row0 + 32 * b, k0, bar);
    }
    if (!p.b.mn_major) {
#pragma unroll
      for (int h = 0; h < KSUB; ++h) ptx::tma_load_2d_pair(b_dst + h * (B_ROWS * 128), &tm_b, k0 + h * (int32_t)p.sub_k, b_row0, bar);
    } else if (!p.tf32) {
#pragma unroll
      for (int b = 0; b < B_ROWS / 64; ++b) ptx::tma_load_2d_pair(b_dst + b * MN_BOX_BYTES, &tm_b, b_row0 + 64 * b, k0, bar);
    } else {
#pragma unroll
      for (int b = 0; b < B_ROWS / 32; ++b) ptx::tma_load_2d_pair(b_dst + b * (MN_BOX_BYTES / 2), &tm_b, b_row0 + 32 * b, k0, bar);
    }
  };
  auto issue_early = [&]() {
    if (ptx::elect_one()) {
      for (int32_t j = 0; j < early; ++j) {
        EXO_TRACE(0, j, 0, 2048);
        issue_loads(j, (uint32_t)j);
        EXO_TRACE(0, j, 1, 2048);
      }
    }
  };

  // ---------------------------------------------------------------- set-up
  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tm_a);
      ptx::prefetch_tensormap(&tm_b);
      ptx::grid_launch_dependents();   // the next kernel's own set-up may overlap this whole kernel
    }
    for (uint32_t i = lane; i < kBarriers; i += 32u) ptx::mbar_init(bar0 + 8u * i, i == 2 * kMaxStages + 1 ? (uint32_t)EW : 1u);
    ptx::fence_mbar_init();
    ptx::fence_proxy_async_smem();     // the copies signal these barriers through the async proxy
    __syncwarp();
    // The operands may be the previous kernel's output; nothing before this line reads global memory.
    ptx::grid_dependency_wait();
    if (cta_rank == 0) issue_early();  // the leader's copies count on its own barriers, which exist now
  } else if (warp == 1) {
    ptx::tmem_alloc<2>(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish<2>();
  } else if (warp == 2 && lane == 0) {
    ptx::prefetch_tensormap(&tm_c);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  // the peer's barriers and tensor memory exist before anything remote touches them: the other CTA's copies
  // (the leader's barriers), the MMAs (the other CTA's shared and tensor memory), the commits (its barriers)
  ptx::cluster_arrive();
  ptx::cluster_wait();
  ptx::tc_fence_after_sync();
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot) : "memory");
  if (warp != 0) ptx::grid_dependency_wait();   // (returns at once: warp 0 passed it before the barriers above)
  if (threadIdx.x == 64) EXO_TRACE(2, 4094, 0, 4096);

  if (warp == 0) {
    // ============================================================ producer
    if (cta_rank != 0) issue_early();
    uint32_t s = (uint32_t)early, ph = 0;
    if (s == (uint32_t)STAGES) { s = 0; ph = 1u; }
    for (int32_t j = early; j < nkb && ok; ++j) {
      if (j >= STAGES) {
        ok = wait_barrier<true>(empty_bar(s), ph ^ 1u, p, WaitSite{kRoleProducer, s, blockIdx.x, (uint32_t)j});
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
    // ============================================================ MMA issuer (leading CTA) and owner of tensor memory
    if (cta_rank == 0) {
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
        ok = wait_barrier<true>(full_bar(s), ph, p, WaitSite{kRoleMma, s, blockIdx.x, (uint32_t)j});
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        if (ptx::elect_one()) {
          EXO_TRACE(1, j, 0, 2048);
          const uint32_t a_addr = stage0 + s * STAGE_BYTES;
          const uint64_t a_desc = make_smem_desc(a_addr, p.a), b_desc = make_smem_desc(a_addr + A_BYTES, p.b);
          const int32_t k_left = p.K - j * STAGE_K;
          if (k_left >= STAGE_K && !tf32) {
#pragma unroll
            for (int32_t k = 0; k < kMmaPerStage; ++k)
              ptx::umma_f16<2>(tmem_base, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc,
                               (j != 0 || k != 0) ? 1u : 0u);
          } else {  // tf32, or a ragged last k-block, which skips the MMAs that would only read zero fill
            const int32_t n_mma = k_left >= STAGE_K ? kMmaPerStage : (k_left + umma_k - 1) / umma_k;
            for (int32_t k = 0; k < n_mma; ++k) {
              const uint32_t accumulate = (j != 0 || k != 0) ? 1u : 0u;
              if (tf32) ptx::umma_tf32<2>(tmem_base, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc, accumulate);
              else ptx::umma_f16<2>(tmem_base, a_desc + k_off(k, a_step, a_sub), b_desc + k_off(k, b_step, b_sub), idesc, accumulate);
            }
          }
          if (j + STAGES < nkb) ptx::umma_commit<2>(empty_bar(s), 3);   // only a stage that is filled again is released, in both CTAs
          if (j == nkb - 1) ptx::umma_commit<2>(tfull_bar, 3);           // accumulator complete, told to both CTAs
          EXO_TRACE(1, j, 1, 2048);
        }
        __syncwarp();
        if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1u; }
      }
    }
    // wait until this CTA's epilogue warps have read the accumulator (they arrive also when they give up)
    const bool drained = wait_barrier<false>(tdone_bar, 0u, p, WaitSite{kRoleMma, 120, blockIdx.x, 0});
    if (!__all_sync(0xffffffffu, drained && ok))
      for (int i = 0; i < 200; ++i) __nanosleep(1000);   // a wait was abandoned: let MMAs in flight land first
    ok = true;   // (the pause after an abandoned wait has been taken)
  } else {
    // ============================================================ epilogue
    const uint32_t ew = warp - 2u;
    const uint32_t quad = warp & 3u;                 // the TMEM lanes a warp may read: 32 * (warp % 4) ..
    const int32_t first_chunk = (int32_t)(ew >> 2) * CPW;
    const int32_t row0 = cta_row0 + (int32_t)quad * 32;
    int32_t mine = 0;                                 // this warp's chunks that hold any valid element
    if (row0 < p.M) {
      const int32_t nch = (p.N - col0 + CW - 1) / CW - first_chunk;
      mine = nch < 0 ? 0 : (nch > CPW ? CPW : nch);
    }
    // a staging buffer per chunk and quadrant in the operand ring, which is idle once the accumulator is complete
    const uint32_t buf0 = stage0 + (quad * NCHUNK + (uint32_t)first_chunk) * kEpiBufBytes;
    const bool has_beta = p.beta != 0.f, has_acc = nkb > 0, scale = p.alpha != 1.f;
    const float alpha = p.alpha, beta = p.beta;
    if (has_acc) {
      ok = wait_barrier<true>(tfull_bar, 0u, p, WaitSite{kRoleEpilogue, 200, blockIdx.x, 0});
      ok = __all_sync(0xffffffffu, ok);
      ptx::tc_fence_after_sync();
    }
    if (warp == 2 && lane == 0) EXO_TRACE(2, 0, 0, 4096);
    if (ok && has_beta && mine > 0 && ptx::elect_one()) {   // C_in of all of this warp's chunks at once
      ptx::mbar_arrive_expect_tx(cin_bar(ew), (uint32_t)mine * kEpiBufBytes);
      for (int32_t i = 0; i < mine; ++i)
        ptx::tma_load_2d(buf0 + (uint32_t)i * kEpiBufBytes, &tm_c, col0 + (first_chunk + i) * CW, row0, cin_bar(ew));
    }
    __syncwarp();
    const uint32_t tacc = tmem_base + ((quad * 32u) << 16);
    const uint32_t my_xor = (lane & 7u) << 4;
    bool cin_ready = !(has_beta && mine > 0);
#pragma unroll 1
    for (int32_t i = 0; i < CPW; ++i) {
      uint32_t v[UPC][32];
      if (ok && has_acc && i < mine) {
#pragma unroll
        for (int q = 0; q < UPC; ++q) ptx::tmem_ld_32x32(tacc + (uint32_t)((first_chunk + i) * CW + q * 32), v[q]);
        ptx::tmem_ld_wait();
      } else {
#pragma unroll
        for (int q = 0; q < UPC; ++q)
#pragma unroll
          for (int k = 0; k < 32; ++k) v[q][k] = 0u;
      }
      EXO_TRACE_CHUNK(i, 1);
      if (i == mine - 1 || (mine == 0 && i == 0)) {   // this warp's last read of the accumulator
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (ptx::elect_one()) ptx::mbar_arrive(tdone_bar);
      }
      if (!ok || i >= mine) continue;
      if (!cin_ready) {
        ok = wait_barrier<false>(cin_bar(ew), 0u, p, WaitSite{kRoleEpilogueCin, 300, blockIdx.x, 0});
        ok = __all_sync(0xffffffffu, ok);
        cin_ready = true;
        if (!ok) continue;
      }
      const uint32_t my_row = buf0 + (uint32_t)i * kEpiBufBytes + lane * 128u;
      auto piece = [&](int j) { return my_row + (((uint32_t)j << 4) ^ my_xor); };   // 128-byte swizzle
#pragma unroll
      for (int q = 0; q < UPC; ++q) {
        uint32_t(&cur)[32] = v[q];
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
    if (ok) {
      // the stores must have read this warp's buffers before the CTA leaves
      if (warp == 2 && lane == 0) EXO_TRACE(2, 0, 1, 4096);
      if (ptx::elect_one()) ptx::bulk_wait_read<0>();
      __syncwarp();
    }
  }
  // A thread that gave up a wait lets copies and MMAs still in flight land before shared and tensor memory go.
  if (!ok)
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  // Both CTAs' shared and tensor memory stay until both are done: the leader's MMAs read the other CTA's
  // stages and write its accumulator, and tensor memory of a pair is freed by the pair.
  ptx::tc_fence_before_sync();
  ptx::cluster_arrive();
  ptx::cluster_wait();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<2>(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0) EXO_TRACE(2, 4095, 1, 4096);
}

}  // namespace exo
