// Primitives for kernels in which the two CTAs of a cluster share every tensor-core MMA
// (tcgen05 cta_group::2): cluster rank and barrier, tensor copies that complete on the leader's barrier,
// the scoped remote mbarrier arrival, bounded waits that
// raise both CTAs' abort flags, paired tensor-memory management, the paired MMA and its multicast
// commit.  No TMA multicast is used anywhere.
#pragma once

#include "tc_common.cuh"

namespace npas {
namespace tc {

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier of another CTA of the cluster with release semantics at cluster scope: what the PTX
// memory model asks for between threads of two CTAs.  It holds the arriving thread for several hundred
// cycles (longer under load; the unscoped form costs about 90), so the pair kernels keep it off the critical
// path: the only such arrival hands an accumulator back, once per output tile.
__device__ __forceinline__ void mbar_arrive_remote_release(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// 2-D tiled load into this CTA's shared memory whose completion is counted on a barrier of the pair's
// leader (cluster address): the form of the tensor copy that may signal the peer CTA's barrier.  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *m, uint32_t bar_cluster_addr, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void st_remote_u32(uint32_t cluster_addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// Bounded wait on a barrier of this CTA that the pair's tensor copies or MMA commits complete; on expiry both
// CTAs' abort flags are raised.  kClusterScope: the acquire is taken at cluster scope, for the one barrier on
// which a THREAD of the other CTA arrives (with release at cluster scope) after it has read tensor memory.
template <bool kClusterScope = false>
__device__ __forceinline__ bool pair_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t peer_abort_addr, uint32_t *ws, uint32_t where)
{
    auto ready = [&]() { return kClusterScope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    if (ready()) return true;
    long long t0 = 0;
    uint32_t spins = 0;
    while (!ready()) {
        __nanosleep(32);
        ++spins;
        if (spins == 256u) t0 = clock64();
        else if ((spins & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                st_remote_u32(peer_abort_addr, 1u);
                if (atomicCAS(ws, 0u, 10u /* NPAS_ERR_TIMEOUT */) == 0u) ws[1] = where;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *slot_in_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(slot_in_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A[smem, 128 rows per CTA] * B[smem, N/2 rows per CTA]; issued by ONE thread of the leader.
__device__ __forceinline__ void mma_bf16_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on the barrier at this offset in both CTAs once every MMA issued so far has completed.
__device__ __forceinline__ void mma_commit_pair(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}


}  // namespace tc
}  // namespace npas
