// Two-CTA variant of the persistent dense GEMM (tcgen05 cta_group::2) for plans whose SM set consists of
// whole TPCs (both SMs of every chosen TPC), e.g. every full-chip plan and every die-compact set.
//
// Two thread blocks form a cluster and compute one 256 x 256 output unit together: block r of
// the pair holds rows [128 r, 128 r + 128) of the A tile and columns [128 r, 128 r + 128) of the
// B tile in its own shared memory, the leader block (rank 0) issues one MMA per K = 16 step for
// both, and every block ends up with its 128 x 256 part of the result in its own tensor memory.
// Per SM a k-slab costs 32 KB of copies instead of 48 KB, which matters because a single SM's
// TMA unit keeps only ~32 KB of copies in flight: the one-CTA kernel waits for data a fifth of
// the time, this one does not.
//
// Pinning (Section 7.1.2 of the paper) works as in the one-CTA kernel: every block reads %smid and
// takes the plan slot of its SM.  The two blocks of a pair tell each other their slots and walk the
// two task lists in alternation, so every list of the plan is still run exactly once.  No copy is
// shared between blocks: each block loads its own halves; only the "stage is free" and "accumulator is
// ready" signals of tcgen05.commit go to both blocks.
#include <string.h>

#include <mutex>

#include "pair.cuh"

namespace ag {

constexpr int P_BM = 128;        // rows per block (256 per pair)
constexpr int P_BN = 256;        // columns of the unit
constexpr int P_BNH = 128;       // B columns held by one block
constexpr int P_BK = 64;         // k-slab
// A stage holds two k-slabs (64 KB per block, 8 MMAs): the thread that issues the MMAs pays a fixed cost per stage
// (barrier wait, fence, commit) that four MMAs did not cover.  A warp gets only about two bulk copies in flight,
// so each of the three stages has its own copy-issuing warp (A and B of its stage: 2 x 32 KB).
constexpr int P_SLABS = 2;
constexpr int P_STAGES = 3;
constexpr int P_NPROD = P_STAGES;
constexpr int P_THREADS = (2 + kEpiWarps + P_NPROD) * 32;   // scheduler, MMA issuer, epilogue warps, copy warps
constexpr int P_A_SLAB = P_BM * P_BK * 2;      // 16 KB
constexpr int P_B_SLAB = P_BK * P_BNH * 2;     // 16 KB
constexpr int P_A_BYTES = P_SLABS * P_A_SLAB;  // 32 KB
constexpr int P_B_BYTES = P_SLABS * P_B_SLAB;  // 32 KB
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES;
constexpr int P_EPI_BUF = 32 * 32 * 4;
constexpr int P_EPI_BYTES = kEpiWarps * 2 * P_EPI_BUF;
constexpr int P_SMEM_BYTES = P_STAGES * P_STAGE_BYTES + P_EPI_BYTES + 1024 + 1024;
constexpr int P_TMEM_COLS = 512;

struct PairCtl {
    uint64_t full[P_STAGES];       // leader's copy collects the bytes of both blocks
    uint64_t empty[P_STAGES];      // signalled in both blocks by the leader's commit
    uint64_t tmem_full[2];         // signalled in both blocks by the leader's commit
    uint64_t tmem_empty[2];        // leader's copy: 8 arrivals (4 epilogue warps of each block)
    uint64_t sched_full[kRing];
    uint64_t sched_empty[kRing];
    uint64_t mma_drain;
    int ring[kRing];
    uint32_t tmem_base;
    int abort_flag;
    int member;
    int peer_slot;                 // written by the other block of the pair
};

// PACKED_B: the B panels come from die-local 4 KB pages ([128 columns x 16 k], no-swizzle core-matrix order,
// see ag_pack_weights): tm_b then describes the packed buffer as [chunk][16][128] and a page is one box.
template <bool PACKED_B>
__global__ void __launch_bounds__(P_THREADS, 1)
k_gemm_persistent_pair(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                       const __grid_constant__ CUtensorMap tm_b2, const __grid_constant__ CUtensorMap tm_c,
                       const PersistParams p, const int32_t* __restrict__ page_table, const int pages_per_block,
                       const int32_t* __restrict__ quad_base, const GroupView gv) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t s_epi = base + P_STAGES * P_STAGE_BYTES;
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem + P_STAGES * P_STAGE_BYTES + P_EPI_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int my_sm = (int)smid();
    const PlanLayout lay{p.b, p.n_units, p.n_sm};

    // take the slot of this SM; a pair on an unplanned TPC has nothing to do and leaves after the hand-shake
    const int slot = p.image[lay.smid_to_slot() + my_sm];
    if (tid == 0) {
        ctl->abort_flag = 0;
        ctl->member = slot >= 0 && atomicMax(&p.claimed[slot], p.epoch) < p.epoch;
        for (int i = 0; i < P_STAGES; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), 2 * kEpiWarps);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&ctl->sched_full[i]), 1);
            mbar_init(smem_u32(&ctl->sched_empty[i]), 1 + kEpiWarps + P_NPROD);
        }
        mbar_init(smem_u32(&ctl->mma_drain), 1);
        mbar_fence_init();
        prefetch_tmap(&tm_a);
        prefetch_tmap(&tm_b);
        prefetch_tmap(&tm_c);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), P_TMEM_COLS);   // all 512 columns: both blocks get the same base
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // both blocks are running and have their barriers set up; then tell the peer which slot this block
    // holds (-1: it has none) and meet again
    cluster_sync();
    if (tid == 0) st_cluster_u32(map_to_cta(smem_u32(&ctl->peer_slot), rank ^ 1u), (uint32_t)(ctl->member ? slot : -1));
    cluster_sync();
    const int peer_slot = ctl->peer_slot;
    const bool active = ctl->member && peer_slot >= 0;
    if (!active && tid == 0 && (ctl->member || peer_slot >= 0))
        atomicCAS(&p.ctrl->status, 0, (int)AG_ERR_UNMANNED_SM);  // half a pair cannot run this kernel
    const uint32_t tmem_base = ctl->tmem_base;
    const uint64_t limit = p.wait_limit_ns;

    if (active) {
        if (warp == 0) {
            // ------------------------------------------------ scheduler: hands the pair's unit sequence to the other roles
            PairSource src(p, slot, peer_slot, gv);
            int ok = 1;
            for (uint32_t it = 0; ok; ++it) {
                const int u = src.next();
                if (lane == 0) {
                    const int r = it % kRing;
                    if (!mbar_wait_idle(smem_u32(&ctl->sched_empty[r]), ((it / kRing) & 1) ^ 1, abort_flag, limit)) {
                        report_timeout(p, 1);
                        ok = 0;
                    } else {
                        ctl->ring[r] = u;
                        if (p.unit_times && u >= 0) p.unit_times[2 * u] = globaltimer_ns();
                        mbar_arrive(smem_u32(&ctl->sched_full[r]));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (u < 0) break;
            }
        } else if (warp >= 2 + kEpiWarps) {
            // ------------------------------------------------ copies: warp pw fills stage pw (its A and its B part).  For
            // packed B the lanes look up the chunks of the stage's pages one stage ahead of the copies.
            const int pw = warp - (2 + kEpiWarps);
            const uint32_t sa = base + pw * P_STAGE_BYTES, sb_addr = sa + P_A_BYTES;
            const uint32_t bar_own = smem_u32(&ctl->full[pw]);
            const uint32_t bar_leader = map_to_cta(bar_own, 0);        // the leader's barrier counts the bytes of both blocks
            const uint32_t bar_empty = smem_u32(&ctl->empty[pw]);
            uint32_t q_run = 0;      // stages (over the whole run of this pair) before the current unit
            int ok = 1;
            for (uint32_t it = 0; ok; ++it) {
                const int r = it % kRing;
                int u = -1;
                if (lane == 0) {
                    if (!mbar_wait_idle(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                        report_timeout(p, 8);
                        ok = 0;
                    } else {
                        u = ctl->ring[r];
                        mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                u = __shfl_sync(0xffffffffu, u, 0);
                if (!ok || u < 0) break;
                const int tm = u / p.tiles_n, tn = u % p.tiles_n;
                const int grp = gv.rows ? tn / gv.tiles_per_group : 0;        // expert of this unit column
                const int tl = gv.rows ? tn - grp * gv.tiles_per_group : tn;  // unit column inside the expert
                const CUtensorMap* ma = gv.rows ? &gv.tm_a[grp] : &tm_a;
                const CUtensorMap* mb = (gv.rows && !PACKED_B) ? &gv.tm_b[grp] : &tm_b;
                const int n_st = (p.kslabs_total + P_SLABS - 1) / P_SLABS;
                // Packed B: the units of one raster group that share a column panel start their k loop at different
                // stages (the sum over k does not care where it starts), so that at any moment they read different
                // 4 KB pages: a page sits in few L2 slices, and eight pairs asking for the same page at once queue up there.
                const int rot = PACKED_B ? ((tm & 7) * max(1, n_st / 8)) % n_st : 0;
                const int i0 = (pw + P_NPROD - (int)(q_run % P_NPROD)) % P_NPROD;   // this warp's first stage of the unit
                uint32_t ph = (((q_run + i0) / P_STAGES) & 1) ^ 1;                  // parity of "stage is free"
                auto table_entry = [&](int i) -> int {
                    if (!PACKED_B || i >= n_st) return 0;
                    const int s = ((i + rot) % n_st) * P_SLABS;
                    const size_t blk = (size_t)(tn * 2 + (int)rank);
                    if (quad_base) return (lane < P_SLABS && s + lane < p.kslabs_total) ? quad_base[blk * (pages_per_block / 4) + s + lane] : 0;
                    return (lane < 4 * P_SLABS && s + (lane >> 2) < p.kslabs_total) ? page_table[blk * pages_per_block + (size_t)s * 4 + lane] : 0;
                };
                int next_entry = table_entry(i0);
                for (int i = i0; i < n_st && ok; i += P_NPROD) {
                    const int entry = next_entry;
                    next_entry = table_entry(i + P_NPROD);
                    const int s = ((i + rot) % n_st) * P_SLABS;          // first k-slab of this stage
                    const int ns = min(P_SLABS, p.kslabs_total - s);
                    if (lane == 0) {
                        if (!mbar_wait(bar_empty, ph, abort_flag, limit)) {
                            report_timeout(p, 2);
                            ok = 0;
                        } else {
                            // row-major operands always arrive as whole boxes (rows past K are zeros)
                            if (leader) mbar_expect_tx(bar_own, 2 * (P_A_BYTES + (PACKED_B ? ns * P_B_SLAB : P_B_BYTES)));
                            if (p.a_blocks) {
                                tma_load_3d_pair(sa, ma, bar_leader, 0, tm * 2 * P_BM + (int)rank * P_BM, s);
                            } else {
                                tma_load_2d_pair(sa, ma, bar_leader, s * P_BK, tm * 2 * P_BM + (int)rank * P_BM);
                                tma_load_2d_pair(sa + P_A_SLAB, ma, bar_leader, (s + 1) * P_BK, tm * 2 * P_BM + (int)rank * P_BM);
                            }
                            if (!PACKED_B) {
                                if (p.b_blocks) {
                                    // both 64-column blocks of this block's half with one copy
                                    tma_load_3d_pair(sb_addr, mb, bar_leader, 0, s * P_BK, tl * 4 + (int)rank * 2);
                                } else {
                                    tma_load_2d_pair(sb_addr, mb, bar_leader, tl * P_BN + (int)rank * P_BNH, s * P_BK);
                                    tma_load_2d_pair(sb_addr + P_B_BYTES / 2, mb, bar_leader, tl * P_BN + (int)rank * P_BNH + 64, s * P_BK);
                                }
                            }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (PACKED_B && quad_base) {
                        // a slab's four pages are one group of same-die chunks: one strided box each
                        if (lane < ns) tma_load_5d_pair(sb_addr + lane * P_B_SLAB, (entry >> 30) ? &tm_b2 : &tm_b, bar_leader, 0, 0, 0, 0, entry & 0x3fffffff);
                    } else if (PACKED_B) {
                        // one lane per 4 KB page, all in one instruction
                        if (lane < 4 * ns) tma_load_3d_pair(sb_addr + lane * 4096, &tm_b, bar_leader, 0, 0, entry);
                    }
                    ph ^= 1;     // the next stage this warp fills is the same buffer, one round later
                }
                q_run += (uint32_t)n_st;
            }
        } else if (warp == 1) {
            {
                // ------------------------------------------------ MMA issuer (leader) / ring consumer (peer)
                // All 32 lanes run the loop converged and one elected lane issues the MMAs and commits (see elect_one).
                constexpr uint32_t idesc = make_idesc_bf16(2 * P_BM, P_BN, 0, PACKED_B ? 0 : 1);
                // descriptors without their start address.  A: K-major, 128-byte swizzle, 8 rows 1 KB apart.  B: row-major
                // source = N-major, 128-byte swizzle, the two 64-column blocks half the B part apart (LBO), 8 k rows 1 KB
                // apart (SBO); packed page = K-major, no swizzle, 16-byte k chunks 128 B apart (LBO), 8-column groups
                // 256 B apart (SBO).  The address field counts 16-byte units and never carries out of its 14 bits.
                const uint64_t da_t = make_smem_desc(0, 16, 1024, 2);
                const uint64_t db_t = PACKED_B ? make_smem_desc(0, 128, 256, 0) : make_smem_desc(0, P_B_BYTES / 2, 1024, 2);
                constexpr uint32_t kAStep = 32u >> 4, kASlabStep = (uint32_t)P_A_SLAB >> 4;
                constexpr uint32_t kBStep = (PACKED_B ? 4096u : 2048u) >> 4;
                const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
                uint32_t st = 0, ph = 0, tile_it = 0;
                bool ok = true;
                for (uint32_t it = 0; ok; ++it) {
                    const int r = it % kRing;
                    if (!mbar_wait_all(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 3);
                        break;
                    }
                    const int u = ctl->ring[r];
                    __syncwarp();       // every lane has read the entry before it is handed back
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                    if (u < 0) break;
                    if (!leader) continue;
                    const uint32_t acc = tile_it & 1;
                    if (!mbar_wait_all(smem_u32(&ctl->tmem_empty[acc]), ((tile_it >> 1) & 1) ^ 1, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 4);
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * P_BN;
                    // the stages arrive in the order the copy warps walk them; with packed B that order is rotated,
                    // but how many k-slabs a stage holds depends only on whether it is the unit's last one in k
                    const int n_st = (p.kslabs_total + P_SLABS - 1) / P_SLABS;
                    const int tm = u / p.tiles_n;
                    const int rot = PACKED_B ? ((tm & 7) * max(1, n_st / 8)) % n_st : 0;
                    const bool odd_tail = (p.kslabs_total & 1) != 0;
                    for (int i = 0; i < n_st; ++i) {
                        if (!mbar_wait_all(full0 + st * 8, ph, abort_flag, limit)) {
                            if (lane == 0) report_timeout(p, 5);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t sa = base + st * P_STAGE_BYTES;
                        const uint64_t da = da_t | (uint64_t)(sa >> 4);
                        const uint64_t db = db_t | (uint64_t)((sa + P_A_BYTES) >> 4);
                        const bool half = odd_tail && ((i + rot) % n_st) == n_st - 1;   // the stage that holds the last, single k-slab
                        if (elect_one()) {
                            tc_mma_f16_pair(d_tmem, da, db, idesc, i > 0 ? 1u : 0u);
#pragma unroll
                            for (int k4 = 1; k4 < P_BK / 16; ++k4) tc_mma_f16_pair(d_tmem, da + k4 * kAStep, db + k4 * kBStep, idesc, 1u);
                            if (!half) {
#pragma unroll
                                for (int k4 = 0; k4 < P_BK / 16; ++k4)
                                    tc_mma_f16_pair(d_tmem, da + kASlabStep + k4 * kAStep, db + (4 + k4) * kBStep, idesc, 1u);
                            }
                            tc_commit_pair(empty0 + st * 8);
                        }
                        __syncwarp();
                        if (++st == P_STAGES) { st = 0; ph ^= 1; }
                    }
                    if (!ok) break;
                    if (elect_one()) tc_commit_pair(smem_u32(&ctl->tmem_full[acc]));
                    __syncwarp();
                    ++tile_it;
                }
                __syncwarp();
                if (leader && *abort_flag) {
                    if (elect_one()) {
                        tc_commit(smem_u32(&ctl->mma_drain));
                        int dummy = 0;
                        mbar_wait(smem_u32(&ctl->mma_drain), 0, &dummy, 2000000ull);
                    }
                    __syncwarp();
                }
            }
        } else {
            // ------------------------------------------------ epilogue warps: this block's 128 rows of the unit
            const int q = warp & 3;
            const uint32_t buf0 = s_epi + (warp - 2) * 2 * P_EPI_BUF;
            uint32_t tile_it = 0, chunk_it = 0;
            for (uint32_t it = 0;; ++it) {
                const int r = it % kRing;
                if (!mbar_wait_warp(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                    if (lane == 0) report_timeout(p, 6);
                    break;
                }
                const int u = ctl->ring[r];
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                if (u < 0) break;
                const int tm = u / p.tiles_n, tn = u % p.tiles_n;
                const uint32_t acc = tile_it & 1;
                if (!mbar_wait_warp(smem_u32(&ctl->tmem_full[acc]), (tile_it >> 1) & 1, abort_flag, limit)) {
                    if (lane == 0) report_timeout(p, 7);
                    break;
                }
                tc_fence_after();
                const int row0 = tm * 2 * P_BM + (int)rank * P_BM + q * 32;
                const int grp = gv.rows ? tn / gv.tiles_per_group : 0;
                const int tl = gv.rows ? tn - grp * gv.tiles_per_group : tn;
                const CUtensorMap* mc = gv.rows ? &gv.tm_c[grp] : &tm_c;
                const int m_rows = gv.rows ? gv.rows[grp] : p.M, n_cols = gv.rows ? gv.n_group : p.N;
#pragma unroll 1
                for (int c = 0; c < P_BN / 32; ++c, ++chunk_it) {
                    uint32_t v[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * P_BN + c * 32, v);
                    tmem_ld_wait();
                    const uint32_t buf = buf0 + (chunk_it & 1) * P_EPI_BUF;
                    if (lane == 0) bulk_wait_read<1>();
                    __syncwarp();
                    const uint32_t rowaddr = buf + lane * 128;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t a = rowaddr + ((j ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v[4 * j]), "r"(v[4 * j + 1]),
                                     "r"(v[4 * j + 2]), "r"(v[4 * j + 3])
                                     : "memory");
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int x = tl * P_BN + c * 32;
                        if (x < n_cols && row0 < m_rows) tma_store_2d(mc, buf, x, row0);
                        bulk_commit();
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    // the leader issues the MMAs for both blocks: it must know that both have read this accumulator
                    mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->tmem_empty[acc]), 0));
                    if (q == 0 && leader) {
                        p.tile_owner[u] = my_sm;
                    if (p.unit_times) p.unit_times[2 * u + 1] = globaltimer_ns();
                        atomicAdd(&p.tile_count[u], 1);
                    }
                }
                ++tile_it;
            }
            if (lane == 0) bulk_wait<0>();
        }
    }
    // nobody leaves while the peer may still signal this block's barriers or read its shared memory
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, P_TMEM_COLS);
    }
}

ag_status gemm_pair_dispatch(const void* A, const void* B, const ag_packed_weights* W, void* Cout, int M, int N, int K,
                             const ag_plan* plan, cudaStream_t stream, const ag_group_desc* grp) {
    const int32_t* h = plan->header;
    if (M != h[H_M] || N != h[H_N] || K != h[H_K]) return AG_ERR_ARG;
    if (h[H_TILE_M] != 2 * P_BM || h[H_TILE_N] != P_BN || h[H_KSPLITS] != 1 || !h[H_STATIC]) return AG_ERR_ARG;
    if (plan->policy.k_unit != P_BK || (K % 8) || (N % 8)) return AG_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)Cout) & 15u) return AG_ERR_ARG;
    if (W) {
        if (W->K != K || W->N != N || (K % P_BK) || W->tiles_n != 2 * h[H_TILES_N]) return AG_ERR_ARG;
    } else if (grp) {
        if (!grp->d_tm_w) return AG_ERR_ARG;
    } else if (!B || ((uintptr_t)B & 15u)) {
        return AG_ERR_ARG;
    }
    if (grp && (!grp->d_tm_c || (grp->N % P_BN))) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    if ((st = refuse_capture(stream)) != AG_OK) return st;
    if ((st = renew_epochs_if_needed(plan, stream)) != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    // A pair of blocks is co-scheduled on the two SMs of one TPC, so the plan must hold whole TPCs: a block
    // whose partner sits on an unplanned SM could not run.  (Seeded random SM subsets do not qualify - the
    // compute-side counterpart of the paper's point that equal SM counts are not equal capabilities.)
    if (n_sm != plan->lay.n_sm || (n_sm & 1) || plan->grid_blocks != 0) return AG_ERR_ARG;  // pairs: always one block per SM
    {
        const int32_t* slot_of = plan->h_image.data() + plan->lay.smid_to_slot();
        for (int s = 0; s < n_sm; ++s)
            if ((slot_of[s] >= 0) != (slot_of[s ^ 1] >= 0)) return AG_ERR_ARG;
    }
    const void* b_key = W ? (const void*)W : B;
    if (grp) {
        if (W) { plan->tm_b = W->quad_free_bit >= 0 ? W->tm_quad[0] : W->tm_pages; plan->tm_b_ptr = nullptr; }
    } else if (plan->tm_a_ptr != A || plan->tm_b_ptr != b_key || plan->tm_c_ptr != Cout) {
        if (!(K % P_BK == 0 ? encode_a_slabs(&plan->tm_a, A, M, K, P_BM, P_SLABS)
                            : encode_2d(&plan->tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, M, K, P_BK, P_BM)))
            return AG_ERR_CUDA;
        if (W) plan->tm_b = W->quad_free_bit >= 0 ? W->tm_quad[0] : W->tm_pages;
        else if (N % 64 == 0) { if (!encode_b_blocks(&plan->tm_b, B, K, N, P_SLABS * P_BK, 2)) return AG_ERR_CUDA; }
        else if (!encode_2d(&plan->tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B, K, N, 64, P_SLABS * P_BK)) return AG_ERR_CUDA;
        if (!encode_2d(&plan->tm_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Cout, M, N, 32, 32)) return AG_ERR_CUDA;
        plan->tm_a_ptr = A; plan->tm_b_ptr = b_key; plan->tm_c_ptr = Cout;
    }
    static std::atomic<unsigned long long> attr_done{0};
    const cudaError_t attr_err = once_per_device(attr_done, [] {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_persistent_pair<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_gemm_persistent_pair<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
        return e;
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err);
    PersistParams gp = make_persist_params(plan, M, N, K);
    gp.b_blocks = grp ? ((!W && grp->w_blocks) ? 1 : 0) : ((!W && N % 64 == 0) ? 1 : 0);
    gp.a_blocks = (!grp && K % P_BK == 0) ? 1 : 0;
    GroupView gv;
    memset(&gv, 0, sizeof gv);
    if (grp) {
        gv.tm_a = grp->d_tm_a; gv.tm_b = grp->d_tm_w; gv.tm_c = grp->d_tm_c; gv.rows = grp->d_rows;
        gv.tiles_per_group = grp->N / P_BN; gv.n_group = grp->N;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(n_sm);
    cfg.blockDim = dim3(P_THREADS);
    cfg.dynamicSmemBytes = P_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int32_t* table = W ? W->d_page_table : nullptr;
    const int32_t* quads = (W && W->quad_free_bit >= 0) ? W->d_quad_base : nullptr;
    const int ppb = W ? W->pages_per_tile : 0;
    const CUtensorMap tm_b2 = quads ? W->tm_quad[1] : plan->tm_b;   // second class of page groups
    const cudaError_t le =
        W ? cudaLaunchKernelEx(&cfg, k_gemm_persistent_pair<true>, plan->tm_a, plan->tm_b, tm_b2, plan->tm_c, gp, table, ppb, quads, gv)
          : cudaLaunchKernelEx(&cfg, k_gemm_persistent_pair<false>, plan->tm_a, plan->tm_b, tm_b2, plan->tm_c, gp, table, ppb, quads, gv);
    if (le != cudaSuccess) return launch_failed(plan, le);
    count_launch();
    return AG_OK;
}

}  // namespace ag
