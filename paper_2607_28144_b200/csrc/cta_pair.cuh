// Helpers for kernels that run on pairs of CTAs (clusters of two, tcgen05 cta_group::2): cluster identity, addresses
// in the other CTA's shared memory, and the paired forms of tensor-memory allocation, tiled load, MMA and commit.
#pragma once
#include <cstdint>

#include "ptx.cuh"

namespace regenvc {

namespace {

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of that barrier, for warps that can do other work in between.
// Arrival of warps that have written nothing the other CTA will read (no release: that fence costs several hundred cycles).
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(n));
    return n;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(n));
    return n;
}
__device__ __forceinline__ uint32_t n_clusters_x() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(n));
    return n;
}
// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
// Whole-warp calls, executed by the same warp of BOTH CTAs of the pair.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Tiled load into THIS CTA's shared memory whose bytes are counted on a barrier that may belong to the other CTA of
// the pair (`bar` is a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const void* tmap, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// D[tensor memory of both CTAs] (+)= A * B over the pair: M = 256 (128 rows of A from each CTA's shared memory),
// N = 256 (128 rows of B from each CTA's shared memory); issued by one thread of the leader CTA.
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on `bar` (a shared::cluster address: this CTA's or the other's) once every pair MMA issued so far by this
// thread has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Arrival on a barrier of either CTA of the pair (shared::cluster address), ordered after this thread's earlier
// accesses at cluster scope.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Arrival on a barrier of either CTA of the pair (shared::cluster address) without cluster-scope ordering of
// ordinary memory: for hand-overs whose payload lives in tensor memory (made visible by tcgen05.wait / fence) or
// is only the fact of the arrival itself.  The cluster-scope release of mbar_arrive_cluster costs hundreds of cycles.
__device__ __forceinline__ void mbar_arrive_peer(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// One 32-bit word from the shared memory of either CTA of the pair (shared::cluster address).
__device__ __forceinline__ uint32_t ld_shared_peer(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
}  // namespace

}  // namespace regenvc
