// Operand sharing between the two CTA pairs of a 4-CTA cluster (single-GPU builds only).
//
// The pairs of a cluster compute neighbouring 256 x BN tiles of the same 256 rows of C, so CTA r
// and CTA r + 2 need the same 128 x K rows of A.  Each of the two fetches 64 of those rows per
// k-block with one TMA load that is multicast to both CTAs: the block crosses the L2-to-SM
// fabric once instead of twice.  This is the "multicast of the shared operand" half of the
// paper's Section 6 cluster kernels, in the form tcgen05 CTA pairs want it:
// with .cta_group::2 the completion bytes of each copy are counted on the mbarrier at the given
// offset in the even (MMA-issuing) CTA of the *receiving* CTA's pair.
//
// The source tensor is always this GPU's own memory.  Never pass a tensor map that covers a peer
// GPU's memory to these functions.
//
// This header is only compiled into the variant library; the base library and every multi-GPU
// run are built without it.
#pragma once
#include <cuda.h>
#include <stdint.h>

namespace exo {

struct SharePairs {
  static constexpr int kPairs = 2;

  // `bar` is the shared::cluster address of the full barrier in an even-ranked CTA; `mask` has one
  // bit per receiving CTA of the cluster.
  static __device__ __forceinline__ void load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y,
                                                 uint32_t bar, uint16_t mask) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "h"(mask)
        : "memory");
  }

  static __device__ __forceinline__ void load_3d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y,
                                                 int32_t z, uint32_t bar, uint16_t mask) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar), "h"(mask)
        : "memory");
  }
};

}  // namespace exo
