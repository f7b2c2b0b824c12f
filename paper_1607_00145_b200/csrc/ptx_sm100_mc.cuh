// Cluster helpers of the CTA-pair variant of the tensor-core kernel: copies that are
// delivered to both CTAs of a pair, and the matching "stage free" signal.  Kept in a file of
// its own (with kernel_umma_mc.cu): runs on more than one GPU are made without them.
// Only this GPU's own memory is ever the source of such a copy.
#pragma once
#include <stdint.h>

namespace ptx_mc {

constexpr uint16_t PAIR_MASK = 3; // both CTAs of the cluster

__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// One box of a tiled tensor map -> the same shared-memory offset in both CTAs of the pair;
// the barrier at offset `bar` of each CTA receives the byte count.
__device__ __forceinline__ void tma_load_pair(uint32_t dst, const void* map, uint32_t bar, int rank, const int32_t* c)
{
    switch (rank) {
    case 2:
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster "
                     "[%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst), "l"(map), "r"(bar), "r"(c[0]), "r"(c[1]),
                     "h"(PAIR_MASK)
                     : "memory");
        break;
    case 3:
        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster "
                     "[%0], [%1, {%3, %4, %5}], [%2], %6;" ::"r"(dst), "l"(map), "r"(bar), "r"(c[0]), "r"(c[1]),
                     "r"(c[2]), "h"(PAIR_MASK)
                     : "memory");
        break;
    case 4:
        asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster "
                     "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(dst), "l"(map), "r"(bar), "r"(c[0]),
                     "r"(c[1]), "r"(c[2]), "r"(c[3]), "h"(PAIR_MASK)
                     : "memory");
        break;
    default:
        asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster "
                     "[%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;" ::"r"(dst), "l"(map), "r"(bar), "r"(c[0]),
                     "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4]), "h"(PAIR_MASK)
                     : "memory");
        break;
    }
}

// The barrier at offset `bar` of BOTH CTAs receives one arrival once all tcgen05 operations
// issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                     bar),
                 "h"(PAIR_MASK)
                 : "memory");
}

} // namespace ptx_mc
