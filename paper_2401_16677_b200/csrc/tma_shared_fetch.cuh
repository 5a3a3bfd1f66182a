// The one TMA load that delivers a tile to more than one CTA of a cluster.  Kept in a file of its own:
// it is compiled only into the single-GPU library variant (macro T3_TMA_SHARED_FETCH, set by the build
// when this file is present), and only ever reads this GPU's own memory (the W operand of the local
// plan).  Everything else in the package builds and runs without this file.
#pragma once
#include <cstdint>

namespace t3 {

// 3-D tiled load for a CTA pair: the box lands at the same shared-memory offset `dst` in every CTA
// named in cta_mask, and each destination's bytes are counted on the barrier at `cluster_bar`'s offset
// in that destination's pair leader.
__device__ __forceinline__ void tma_load_3d_pair_shared(uint32_t dst, const void* tmap, uint32_t cluster_bar, int c0,
                                                        int c1, int c2, uint16_t cta_mask) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
        " [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "h"(cta_mask)
        : "memory");
}

// The same with an L2 eviction-priority policy for the fetched lines.
__device__ __forceinline__ void tma_load_3d_pair_shared_hint(uint32_t dst, const void* tmap, uint32_t cluster_bar, int c0,
                                                             int c1, int c2, uint16_t cta_mask, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
        ".L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6, %7;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "h"(cta_mask),
          "l"(policy)
        : "memory");
}

}  // namespace t3
