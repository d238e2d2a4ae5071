// Helpers shared by the kernels that run a work unit on a pair of thread blocks (tcgen05 cta_group::2, the two SMs of a
// TPC): cluster addressing, copies whose completion is counted by a barrier of the leader block, MMAs and commits of
// the pair, and the unit sequence of a pair.  No copy is shared between blocks (no multicast loads): each block loads
// its own parts; only the arrival of a tcgen05.commit is delivered to both blocks.
#pragma once
#include "persist.cuh"

namespace ag {

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// copy into this block's shared memory, completion bytes reported to a barrier that may sit in the peer block
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int x, int y,
                                                 int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int c0, int c1,
                                                 int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on the barrier at this offset in both blocks of the pair once the MMAs issued so far are done (one
// commit whose arrival is delivered to both blocks; two separate commits cost 7 % at full clock)
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(mask)
        : "memory");
}

// Grouped (MoE-shaped) operation: the plan's N is G experts side by side (expert g = unit columns
// [g * tiles_per_group, (g + 1) * tiles_per_group)), its M the largest row count; every expert has its own
// A, B and C.  All pointers null / 0 for a single problem.
struct GroupView {
    const CUtensorMap* tm_a;   // device [G]
    const CUtensorMap* tm_b;   // device [G] (row-major weights; unused with packed B)
    const CUtensorMap* tm_c;   // device [G]
    const int* rows;           // device [G]
    int tiles_per_group;       // 256-column units per expert
    int n_group;               // columns of one expert
};

// Unit sequence of a pair: the two task lists in alternation, the lower slot first.  In grouped operation
// units that lie below an expert's last row are skipped here, so no role ever sees them.
struct PairSource {
    const int32_t* image;
    const int* g_rows;
    int tiles_per_group, tiles_n;
    int off[2], len[2], pos;
    __device__ PairSource(const PersistParams& p, int slot_a, int slot_b, const GroupView& gv)
        : image(p.image), g_rows(gv.rows), tiles_per_group(gv.tiles_per_group), tiles_n(p.tiles_n), pos(0) {
        const PlanLayout lay{p.b, p.n_units, p.n_sm};
        const int lo = min(slot_a, slot_b), hi = max(slot_a, slot_b);
        off[0] = lay.sm_q() + p.image[lay.sm_q_off() + lo];
        len[0] = p.image[lay.sm_q_off() + lo + 1] - p.image[lay.sm_q_off() + lo];
        off[1] = lay.sm_q() + p.image[lay.sm_q_off() + hi];
        len[1] = p.image[lay.sm_q_off() + hi + 1] - p.image[lay.sm_q_off() + hi];
    }
    __device__ int next() {
        const int common = 2 * min(len[0], len[1]);
        while (true) {
            int u = -1;
            if (pos < common) {
                u = image[off[pos & 1] + (pos >> 1)];
            } else {
                const int longer = len[0] >= len[1] ? 0 : 1;
                const int i = (common >> 1) + (pos - common);
                if (i < len[longer]) u = image[off[longer] + i];
            }
            ++pos;
            if (u < 0 || !g_rows) return u;
            const int tm = u / tiles_n, g = (u % tiles_n) / tiles_per_group;
            if (tm * 2 * 128 < g_rows[g]) return u;   // the expert has rows in this unit row
        }
    }
};

}  // namespace ag
