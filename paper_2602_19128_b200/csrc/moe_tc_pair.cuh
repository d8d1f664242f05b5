// PTX wrappers shared by the CTA-pair (cta_group::2) grouped-GEMM kernels, bf16 and MX FP8.
#pragma once

#include "moe_tc_common.cuh"

namespace moe {
namespace tc {

// Every CTA-pair kernel asks for ALL of an SM's shared memory, whatever its ring needs, so that it never shares an SM
// with another block.  Found the hard way: with a few KiB left over (a 216 KiB ring), small blocks of ANOTHER stream's
// call (the sort-scatter's one-warp blocks, 1 KiB of shared memory each) were scheduled next to pair CTAs, and on two
// streams a later pair on that TPC then waited in tcgen05.alloc for ever -- about once per thousand calls, with every
// pair kernel that left room, the 128-row instance included; with the SM to themselves the same kernels ran tens of
// thousands of overlapping calls.  The cause inside the hardware was not established; exclusivity is what the
// library's pair kernels now guarantee by construction.
constexpr int kPairDynamicSmemBytes = 232448;  // the opt-in maximum: no other block fits (each needs 1 KiB reserved)

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The same arrival without release semantics: for hand-backs that order nothing but tensor-memory reads, which
// tcgen05.wait::ld has already completed.  (A release at cluster scope makes the arriving thread wait until its
// earlier global stores are visible to the peer SM; the epilogue would then drain its stores at every hand-back.)
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void store_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// TMA copies whose completion is signalled on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                                 int c4, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}
// Arrive, on the barrier at this offset in BOTH CTAs, once the MMAs issued so far have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(both)
                 : "memory");
}
// Release of a CTA pair's tensor memory, as the last act of both CTAs.  The deallocation is a collective of the two
// CTAs; each must still be there when the other makes its half of it, so a cluster barrier FOLLOWS it as well as
// precedes it.  (Found with two streams running wide-tile GEMMs: a CTA delayed between the barrier and its
// deallocation -- other streams' small blocks may share its SM -- while its peer had already left, exited with its
// columns still allocated; the next pair on that TPC then waited in tcgen05.alloc for ever.)
__device__ __forceinline__ void tmem_release_pair(uint32_t tmem_base, uint32_t n_cols, int warp) {
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(n_cols) : "memory");
    }
    __syncthreads();
    cluster_sync_all();
}
// Bounded wait that also raises the peer's abort flag when it expires.
__device__ __forceinline__ bool pair_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t peer_abort,
                                          int *status, int site) {
    const bool ok = mbar_wait(bar, parity, abort_flag, status, site);
    if (!ok) store_cluster_u32(peer_abort, 1u);
    return ok;
}

}  // namespace tc
}  // namespace moe
