// Decode-shaped (skinny) persistent GEMM: C[M x N] = A[M x K] * B[K x N] with M <= 32.  The
// weights B are the work: every unit streams a 128-column weight tile over a run of k-slabs, so
// the kernel is HBM bound.  The MMA is turned around: the weight tile is the M = 128 operand,
// the activations are the N = 16 or 32 operand, D[n][m] accumulates in tensor memory.
//
// Weights come either row-major (K x N, consumed in place as an MN-major operand through TMA) or
// packed by ag_pack_weights: 4 KB pages of [128 n x 16 k] elements, each page already in the
// MMA's no-swizzle core-matrix order and stored in a chunk of the die that owns its work unit
// (indirect allocation by remapping, Section 7.1.1 of the paper).  A packed page is fetched with
// one 4 KB bulk copy whose source address comes from the page table.
//
// Split-K units write partial sums to a scratch workspace; the block that completes a tile's
// last split adds them in ascending split order (deterministic) and writes C.
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>

#include "persist.cuh"

namespace ag {

constexpr int SK_BN = 128;     // weight columns per unit
constexpr int SK_BK = 64;      // k-slab
// Six stages (about 110 KB in flight per SM) already cover bandwidth x latency several times; a deeper
// ring only lengthens the queues in the memory system, and with them every dependent round trip
// (fence, arrival atomic, reduction loads).
constexpr int SK_STAGES = 6;
constexpr int SK_W_BYTES = SK_BN * SK_BK * 2;      // 16 KB of weights per stage
constexpr int SK_A_BYTES = 32 * SK_BK * 2;         // room for 32 activation rows
constexpr int SK_STAGE_BYTES = SK_W_BYTES + SK_A_BYTES;
constexpr int SK_SMEM_BYTES = SK_STAGES * SK_STAGE_BYTES + 1024 + 1024;
// An MMA with so few columns finishes its arithmetic in a few cycles but a following MMA that adds to the
// same accumulator has to wait for its result (measured: ~370 cycles per dependent K=16 step).  The
// k-steps of a unit therefore rotate over SK_ACCS independent accumulators, summed in the epilogue.
constexpr int SK_ACCS = 8;

struct SkinnyCtl {
    uint64_t full[SK_STAGES];
    uint64_t empty[SK_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t sched_full[kRing];
    uint64_t sched_empty[kRing];
    uint64_t mma_drain;
    int ring[kRing];
    uint32_t tmem_base;
    int abort_flag;
    int member;
};

struct SkinnyArgs {
    const uint8_t* packed;        // packed weights base (PACKED) or null
    const int32_t* page_table;    // device (PACKED)
    const int32_t* quad_base;     // device (PACKED, grouped layout): first chunk of each k-slab's group, or null
    int quad_f;                   // chunk distance 2^free_bit between the two halves of a group
    int pages_per_tile;
    float* C;
    float* partial;               // [k_splits][M][N] or null when k_splits == 1
    int* sem;                     // [tiles_n * 4]: one arrival counter per 32-column quarter of a tile
    // grouped (MoE-shaped) operation: the plan's N is G experts side by side, expert g = column tiles
    // [g * tiles_per_group, (g + 1) * tiles_per_group); null / 0 when there is a single problem
    const CUtensorMap* g_tm_a;    // device [G]: activations of expert g (rows of the stacked A)
    const CUtensorMap* g_tm_w;    // device [G]: row-major weights of expert g (not PACKED)
    const int* g_rows;            // device [G]
    const int* g_row_off;         // device [G]
    int tiles_per_group;
    int n_group;                  // columns of one expert
};

// Where the output rows of column tile tn live: single problem = C itself; grouped = rows of expert g in the
// stacked C (row stride = columns of one expert).
struct OutView {
    float* base;      // element (row 0, column 0 of the tile's problem)
    int rows;         // valid rows
    int ld;           // row stride in elements
    int col0;         // first column of tile tn inside its problem
    int n_cols;       // columns of the problem
};
__device__ __forceinline__ OutView out_view(const PersistParams& p, const SkinnyArgs& x, int tn) {
    OutView v;
    if (x.g_rows) {
        const int g = tn / x.tiles_per_group, tl = tn - g * x.tiles_per_group;
        v.base = x.C + (size_t)x.g_row_off[g] * x.n_group;
        v.rows = x.g_rows[g];
        v.ld = x.n_group;
        v.col0 = tl * SK_BN;
        v.n_cols = x.n_group;
    } else {
        v.base = x.C; v.rows = p.M; v.ld = p.N; v.col0 = tn * SK_BN; v.n_cols = p.N;
    }
    return v;
}

template <int NM, bool PACKED>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_skinny(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
              const __grid_constant__ CUtensorMap tm_w2, const PersistParams p, const SkinnyArgs x) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    SkinnyCtl* ctl = reinterpret_cast<SkinnyCtl*>(smem + SK_STAGES * SK_STAGE_BYTES);
    constexpr uint32_t kAccCols = SK_ACCS * NM;          // columns of one accumulator set
    constexpr uint32_t kTmemCols = 2 * kAccCols;         // two sets: 256 (NM = 16) or 512 (NM = 32) columns
    volatile int* abort_flag = &ctl->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int my_sm = (int)smid();
    if (tid == 0) ctl->abort_flag = 0;
    const int slot = join_plan(p, &ctl->member);
    if (slot < 0) return;

    if (tid == 0) {
        for (int i = 0; i < SK_STAGES; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), kEpiWarps);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&ctl->sched_full[i]), 1);
            mbar_init(smem_u32(&ctl->sched_empty[i]), 1 + kEpiWarps);
        }
        mbar_init(smem_u32(&ctl->mma_drain), 1);
        mbar_fence_init();
        prefetch_tmap(&tm_a);
        if (!PACKED || x.quad_base) prefetch_tmap(&tm_w);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const uint64_t limit = p.wait_limit_ns;
    constexpr uint32_t kTxBytes = SK_W_BYTES + NM * SK_BK * 2;

    if (warp == 0) {
        // ------------------------------------------------ scheduler + producer.  Lane 0 waits and issues
        // the copies; for packed weights all 32 lanes fetch the page-table entries of the next eight
        // k-slabs (32 pages) with one load each, so the issuing lane never waits on a table lookup.
        UnitSource src(p, slot);
        const uint64_t stream_policy = l2_policy_evict_first();  // weights are read once: do not keep them in L2
        uint32_t it = 0, kit = 0;
        int ok = 1;
        while (ok) {
            const int u = src.next(lane);
            if (lane == 0) {
                const int r = it % kRing;
                if (!mbar_wait(smem_u32(&ctl->sched_empty[r]), ((it / kRing) & 1) ^ 1, abort_flag, limit)) {
                    report_timeout(p, 1);
                    ok = 0;
                } else {
                    ctl->ring[r] = u;
                    if (p.unit_times && u >= 0) p.unit_times[2 * u] = globaltimer_ns();
                    mbar_arrive(smem_u32(&ctl->sched_full[r]));
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ++it;
            if (!ok || u < 0) break;
            const int ks = u % p.k_splits, tn = (u / p.k_splits) % p.tiles_n;
            const int grp = x.tiles_per_group ? tn / x.tiles_per_group : 0;      // expert of this column tile
            const int tl = x.tiles_per_group ? tn - grp * x.tiles_per_group : tn;  // tile inside the expert
            const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
            const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
            for (int sb = s0; sb < s1 && ok; sb += 8) {
                int my_page = 0;
                if (PACKED) {
                    if (x.quad_base) {   // one entry per k-slab: lanes 0..7 fetch the bases of the next eight slabs
                        if (lane < 8 && sb + lane < s1) my_page = x.quad_base[(size_t)tn * (x.pages_per_tile / 4) + sb + lane];
                    } else {
                        const int pg = sb * 4 + lane;
                        if (pg < s1 * 4) my_page = x.page_table[(size_t)tn * x.pages_per_tile + pg];
                    }
                }
                const int se = min(s1, sb + 8);
                for (int s = sb; s < se; ++s, ++kit) {
                    const int st = kit % SK_STAGES;
                    const uint32_t bar = smem_u32(&ctl->full[st]);
                    const uint32_t sw = base + st * SK_STAGE_BYTES, sa = sw + SK_W_BYTES;
                    if (lane == 0) {
                        if (!mbar_wait(smem_u32(&ctl->empty[st]), ((kit / SK_STAGES) & 1) ^ 1, abort_flag, limit)) {
                            report_timeout(p, 2);
                            ok = 0;
                        } else {
                            mbar_expect_tx(bar, kTxBytes);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (PACKED && x.quad_base) {
                        // grouped layout: the slab's four pages sit in chunks q, q+a, q+F, q+F+a of one die
                        // (a = 3 or 1 by q mod 4): one strided box brings all 16 KB
                        const int q0 = __shfl_sync(0xffffffffu, my_page, s - sb);   // bit 30: class of the group
                        if (lane == 0)
                            tma_load_5d_hint(sw, (q0 >> 30) ? &tm_w2 : &tm_w, bar, 0, 0, 0, 0, q0 & 0x3fffffff, stream_policy);
                    } else if (PACKED) {
                        // four lanes issue the four page copies of the slab in one instruction (a single thread
                        // gets only one bulk copy out every ~150 cycles)
                        const int page = __shfl_sync(0xffffffffu, my_page, (s - sb) * 4 + (lane & 3));
                        if (lane < 4)
                            bulk_load_hint(sw + lane * 4096, x.packed + (size_t)page * AG_CHUNK_BYTES, 4096, bar, stream_policy);
                    } else if (lane == 0) {
                        const CUtensorMap* mw = x.g_tm_w ? &x.g_tm_w[grp] : &tm_w;
                        if (p.b_blocks) {
                            // both 64-column blocks with one copy (B seen as [N/64][K][64])
                            tma_load_3d_hint(sw, mw, bar, 0, s * SK_BK, tl * 2, stream_policy);
                        } else {
                            tma_load_2d_hint(sw, mw, bar, tl * SK_BN, s * SK_BK, stream_policy);
                            tma_load_2d_hint(sw + 8192, mw, bar, tl * SK_BN + 64, s * SK_BK, stream_policy);
                        }
                    }
                    if (lane == 0) tma_load_2d(sa, x.g_tm_a ? &x.g_tm_a[grp] : &tm_a, bar, s * SK_BK, 0);
                }
            }
        }
        if (!ok && lane == 0) {
            // gave up: let the copies already in flight land before the block leaves
            const uint32_t n_out = kit < (uint32_t)SK_STAGES ? kit : (uint32_t)SK_STAGES;
            for (uint32_t j = 0; j < n_out; ++j) {
                const uint32_t k2 = kit - 1 - j;
                int dummy = 0;
                mbar_wait(smem_u32(&ctl->full[k2 % SK_STAGES]), (k2 / SK_STAGES) & 1, &dummy, 2000000ull);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, NM, PACKED ? 0 : 1, 0);
            uint32_t kit = 0, tile_it = 0;
            bool ok = true;
            for (uint32_t it = 0; ok; ++it) {
                const int r = it % kRing;
                if (!mbar_wait(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                    report_timeout(p, 3);
                    break;
                }
                const int u = ctl->ring[r];
                mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                if (u < 0) break;
                const int ks = u % p.k_splits;
                const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
                const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
                const uint32_t acc = tile_it & 1;
                if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), ((tile_it >> 1) & 1) ^ 1, abort_flag, limit)) {
                    report_timeout(p, 4);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                for (int s = s0; s < s1; ++s, ++kit) {
                    const int st = kit % SK_STAGES;
                    if (!mbar_wait(smem_u32(&ctl->full[st]), (kit / SK_STAGES) & 1, abort_flag, limit)) {
                        report_timeout(p, 5);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sw = base + st * SK_STAGE_BYTES, sa = sw + SK_W_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < SK_BK / 16; ++k4) {
                        // weights: packed page = no swizzle, 16-byte k chunks 128 B apart (LBO), 8-row groups
                        // 256 B apart (SBO); row-major = MN-major, 128-byte swizzle, as B in the dense kernel
                        const uint64_t dw = PACKED ? make_smem_desc(sw + k4 * 4096, 128, 256, 0)
                                                   : make_smem_desc(sw + k4 * 2048, 8192, 1024, 2);
                        const uint64_t da = make_smem_desc(sa + k4 * 32, 16, 1024, 2);
                        const int step = (s - s0) * 4 + k4;  // k-step of this unit -> accumulator step mod SK_ACCS
                        tc_mma_f16(d_tmem + (step & (SK_ACCS - 1)) * NM, dw, da, idesc, step >= SK_ACCS ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&ctl->empty[st]));
                }
                if (!ok) break;
                tc_commit(smem_u32(&ctl->tmem_full[acc]));
                ++tile_it;
            }
            if (*abort_flag) {
                tc_commit(smem_u32(&ctl->mma_drain));
                int dummy = 0;
                mbar_wait(smem_u32(&ctl->mma_drain), 0, &dummy, 2000000ull);
            }
        }
    } else {
        // ------------------------------------------------ epilogue: lane = weight column n, registers = rows m
        // Split-K hand-off, software-pipelined so that no memory round trip sits between two units:
        //   unit i    its partial sums are stored;
        //   unit i-1  (stores acknowledged long ago) fence, then the arrival counter of its 32 columns
        //             is bumped with an atomic whose result is not looked at yet;
        //   unit i-2  the atomic's result is read: the warp that completed the last of the k_splits
        //             partial sums adds them in ascending split order and writes C.
        // Each epilogue warp owns 32 columns of a tile and its own counter; no barrier between warps.
        const int q = warp & 3;
        uint32_t tile_it = 0, it = 0;
        int st_tn = -1;              // unit whose partial sums are stored but not yet announced
        int at_tn = -1;              // unit whose arrival atomic is in flight
        int oldA = 0, oldB = 0;      // results of the arrival atomics (lane 0), used one unit later
        bool zero_done = false;      // in-memory split-K: the zeroing of C is known to be complete

        auto reduce_columns = [&](int tn) {
            __threadfence();
            // lane = (row group lane/8, four columns); the k_splits loads of one output quad are in flight
            // together and are added in ascending split order
            const int nq = tn * SK_BN + q * 32 + (lane & 7) * 4;
            const OutView ov = out_view(p, x, tn);
            const int nlq = ov.col0 + q * 32 + (lane & 7) * 4;
            if (nq < p.N && nlq < ov.n_cols) {
                for (int m = lane >> 3; m < ov.rows; m += 4) {
                    float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int k0 = 0; k0 < p.k_splits; k0 += 16) {
                        float4 t[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k)
                            if (k0 + k < p.k_splits)
                                t[k] = __ldcg(reinterpret_cast<const float4*>(
                                    x.partial + ((size_t)(k0 + k) * p.M + m) * p.N + nq));
#pragma unroll
                        for (int k = 0; k < 16; ++k)
                            if (k0 + k < p.k_splits) {
                                acc4.x += t[k].x; acc4.y += t[k].y; acc4.z += t[k].z; acc4.w += t[k].w;
                            }
                    }
                    *reinterpret_cast<float4*>(ov.base + (size_t)m * ov.ld + nlq) = acc4;
                }
            }
            __syncwarp();
            if (lane == 0) x.sem[tn * 4 + q] = 0;  // ready for the next launch
        };
        // announce the stored unit (atomic result lands in old_new), resolve the one announced before
        auto hand_off = [&](int& old_use, int& old_new) {
            const int announce = st_tn, resolve = at_tn;
            if (announce >= 0) {
                __threadfence();
                __syncwarp();
                if (lane == 0)
                    asm volatile("atom.global.add.u32 %0, [%1], 1;" : "=r"(old_new) : "l"(x.sem + announce * 4 + q) : "memory");
            }
            if (resolve >= 0) {
                const int last = __shfl_sync(0xffffffffu, old_use == p.k_splits - 1, 0);
                if (last) reduce_columns(resolve);
            }
            at_tn = announce;
            st_tn = -1;
        };
        // one unit; returns false when the list is finished (or a wait ran out)
        auto one_unit = [&](int& old_use, int& old_new) -> bool {
            const int r = it % kRing;
            if (!mbar_wait(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 6);
                return false;
            }
            const int u = ctl->ring[r];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
            ++it;
            if (u < 0) return false;
            const int ks = u % p.k_splits, tn = (u / p.k_splits) % p.tiles_n;
            const uint32_t acc = tile_it & 1;
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), (tile_it >> 1) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 7);
                return false;
            }
            tc_fence_after();
            // sum the accumulators that this unit used
            const int s0e = min(p.kslabs_total, ks * p.kslabs_per_split);
            const int s1e = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
            const int n_used = min(SK_ACCS, (s1e - s0e) * 4);
            float sum[NM];
#pragma unroll
            for (int m = 0; m < NM; ++m) sum[m] = 0.f;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kAccCols;
            for (int j = 0; j < n_used; ++j) {
                uint32_t v[NM];
                if constexpr (NM == 16) tmem_ld_32x16(taddr + j * NM, v); else tmem_ld_32x32(taddr + j * NM, v);
                tmem_ld_wait();
#pragma unroll
                for (int m = 0; m < NM; ++m) sum[m] += __uint_as_float(v[m]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
            ++tile_it;
            const int n = tn * SK_BN + q * 32 + lane;     // column in the plan's (possibly grouped) N
            const OutView ov = out_view(p, x, tn);
            const int nl = ov.col0 + q * 32 + lane;       // column inside the tile's problem
            if (p.k_splits > 1 && x.partial == nullptr) {
                // in-memory reduction: C is zeroed by the kernel launched just before this one, every unit adds
                // its partial sums with reductions that L2 carries out; nothing comes back, so nothing is
                // waited for.  This kernel may have started while the zeroing was still running (programmatic
                // dependent launch): make sure it is complete before the first add.
                if (!zero_done) {
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    zero_done = true;
                }
                if (nl < ov.n_cols) {
#pragma unroll
                    for (int m = 0; m < NM; ++m)
                        if (m < ov.rows) atomicAdd(ov.base + (size_t)m * ov.ld + nl, sum[m]);
                }
            } else if (p.k_splits > 1) {
                hand_off(old_use, old_new);
                float* out = x.partial + (size_t)ks * p.M * p.N;   // workspace rows: the plan's M bound, columns: the plan's N
                if (n < p.N) {
#pragma unroll
                    for (int m = 0; m < NM; ++m)
                        if (m < p.M) out[(size_t)m * p.N + n] = sum[m];
                }
                st_tn = tn;
            } else if (nl < ov.n_cols) {
#pragma unroll
                for (int m = 0; m < NM; ++m)
                    if (m < ov.rows) ov.base[(size_t)m * ov.ld + nl] = sum[m];
            }
            if (lane == 0 && q == 0) {
                p.tile_owner[u] = my_sm;
                    if (p.unit_times) p.unit_times[2 * u + 1] = globaltimer_ns();
                atomicAdd(&p.tile_count[u], 1);
            }
            return true;
        };
        // two copies of the step with the roles of oldA / oldB swapped: the atomic's result register is
        // never copied, so nothing waits for it before the step that needs it
        int which = 0;
        while (true) {
            if (!one_unit(oldA, oldB)) { which = 0; break; }
            if (!one_unit(oldB, oldA)) { which = 1; break; }
        }
        if (p.k_splits > 1 && x.partial != nullptr && !*abort_flag) {
            // drain: `which` = 0 means the atomic in flight wrote oldA (next result goes to oldB)
            if (which == 0) { hand_off(oldA, oldB); hand_off(oldB, oldA); }
            else            { hand_off(oldB, oldA); hand_off(oldA, oldB); }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Zeroes C for the in-memory split-K mode.  Its dependents (the GEMM launched right after it) are released at
// once, so the GEMM's start-up overlaps the zeroing; the GEMM waits for this kernel only before its first add.
__global__ void k_zero_f32(float4* __restrict__ p, size_t n_vec) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x)
        p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// One block per logical page: gathers W[n][k] = B[k][n] for 128 n x 16 k and writes the 4 KB page in
// core-matrix order into its chunk.
__global__ void k_pack_weights(const uint16_t* __restrict__ B, int K, int N, int pages_per_tile,
                               const int32_t* __restrict__ page_table, uint8_t* __restrict__ dst) {
    const int page = blockIdx.x;
    const int tn = page / pages_per_tile, k16 = page % pages_per_tile;
    const int n_local = threadIdx.x;  // 128 threads
    const int n = tn * SK_BN + n_local;
    uint16_t v[16];
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
        const int k = k16 * 16 + kk;
        v[kk] = (n < N && k < K) ? B[(size_t)k * N + n] : (uint16_t)0;
    }
    uint8_t* out = dst + (size_t)page_table[page] * AG_CHUNK_BYTES + (n_local / 8) * 256 + (n_local % 8) * 16;
    uint4 lo, hi;
    lo.x = v[0] | (v[1] << 16); lo.y = v[2] | (v[3] << 16); lo.z = v[4] | (v[5] << 16); lo.w = v[6] | (v[7] << 16);
    hi.x = v[8] | (v[9] << 16); hi.y = v[10] | (v[11] << 16); hi.z = v[12] | (v[13] << 16); hi.w = v[14] | (v[15] << 16);
    *reinterpret_cast<uint4*>(out) = lo;
    *reinterpret_cast<uint4*>(out + 128) = hi;
}

template <int NM, bool PACKED>
static ag_status launch_skinny(const ag_plan* plan, const CUtensorMap& tm_a, const CUtensorMap& tm_w, const CUtensorMap& tm_w2,
                               const PersistParams& gp, const SkinnyArgs& x, cudaStream_t stream, bool after_zeroing) {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(k_gemm_skinny<NM, PACKED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        SK_SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(plan->grid_blocks > 0 ? plan->grid_blocks : plan->lay.n_sm);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SK_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_zeroing ? 1 : 0;   // may start while the zeroing kernel before it is still running
    AG_CUDA(cudaLaunchKernelEx(&cfg, k_gemm_skinny<NM, PACKED>, tm_a, tm_w, tm_w2, gp, x));
    count_launch();
    return AG_OK;
}

// Shared host path of the two skinny entry points.
ag_status gemm_skinny_dispatch(const void* A, const void* B_rowmajor, const ag_packed_weights* W, void* Cout, int M,
                               int N, int K, const ag_plan* plan, float* partial, int* sem, cudaStream_t stream,
                               const ag_group_desc* grp) {
    const int32_t* h = plan->header;
    if (M != h[H_M] || N != h[H_N] || K != h[H_K]) return AG_ERR_ARG;
    if (h[H_TILE_N] != SK_BN || (h[H_TILE_M] != 16 && h[H_TILE_M] != 32) || M > h[H_TILE_M]) return AG_ERR_ARG;
    if (plan->policy.k_unit != SK_BK || (K % 8) || (N % 8)) return AG_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)Cout) & 15u) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (n_sm != plan->lay.n_sm) return AG_ERR_ARG;
    const int NM = h[H_TILE_M];
    CUtensorMap tm_a, tm_w, tm_w2;
    memset(&tm_w, 0, sizeof tm_w);
    memset(&tm_w2, 0, sizeof tm_w2);
    memset(&tm_a, 0, sizeof tm_a);
    if (!grp && !encode_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, M, K, SK_BK, NM)) return AG_ERR_CUDA;
    SkinnyArgs x;
    memset(&x, 0, sizeof x);
    if (grp) {
        x.g_tm_a = grp->d_tm_a;
        x.g_tm_w = W ? nullptr : grp->d_tm_w;
        x.g_rows = grp->d_rows;
        x.g_row_off = grp->d_row_off;
        x.tiles_per_group = grp->N / SK_BN;
        x.n_group = grp->N;
    }
    x.C = (float*)Cout;
    x.partial = h[H_KSPLITS] > 1 ? partial : nullptr;
    x.sem = sem;
    if (W) {
        if (W->K != K || W->N != N || (K % SK_BK) || W->tiles_n != h[H_TILES_N]) return AG_ERR_ARG;
        x.packed = W->dst;
        x.page_table = W->d_page_table;
        x.pages_per_tile = W->pages_per_tile;
        if (W->quad_free_bit >= 0) {
            x.quad_base = W->d_quad_base;
            x.quad_f = 1 << W->quad_free_bit;
            tm_w = W->tm_quad[0];
            tm_w2 = W->tm_quad[1];
        }
    } else if (grp) {
        if (!grp->d_tm_w) return AG_ERR_ARG;  // the descriptor was made without row-major weights
    } else {
        if (!B_rowmajor || ((uintptr_t)B_rowmajor & 15u)) return AG_ERR_ARG;
        if (N % 64 == 0) {
            if (!encode_b_blocks(&tm_w, B_rowmajor, K, N, SK_BK, 2)) return AG_ERR_CUDA;
        } else if (!encode_2d(&tm_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B_rowmajor, K, N, 64, SK_BK)) {
            return AG_ERR_CUDA;
        }
    }
    const bool zeroing = h[H_KSPLITS] > 1 && !x.partial;
    if (zeroing) {  // in-memory reduction mode: the adds need a zeroed C (N % 8 == 0 and 16-byte alignment: whole float4s)
        const size_t c_elems = grp ? (size_t)grp->total_rows * (size_t)grp->N : (size_t)M * (size_t)N;
        const size_t n_vec = c_elems / 4;
        const unsigned blocks = (unsigned)std::min<size_t>(148, (n_vec + 255) / 256);
        k_zero_f32<<<blocks, 256, 0, stream>>>((float4*)Cout, n_vec);
        count_launch();
        AG_CUDA(cudaGetLastError());
    }
    PersistParams gp = make_persist_params(plan, M, N, K);
    gp.b_blocks = grp ? ((!W && grp->w_blocks) ? 1 : 0) : ((!W && N % 64 == 0) ? 1 : 0);
    if (NM == 16) return W ? launch_skinny<16, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, zeroing)
                           : launch_skinny<16, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, zeroing);
    return W ? launch_skinny<32, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, zeroing)
             : launch_skinny<32, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, zeroing);
}

}  // namespace ag

using namespace ag;

// Packs G source matrices (K x n_src each, row-major) side by side: the plan's N is G * n_src.  G = 1 is the
// plain case.
static ag_status pack_weights_impl(const void* const* B_list, int G, int K, int N, const ag_plan* plan,
                                   const ag_affinity_map* amap, void* dst, size_t dst_bytes, uint32_t flags,
                                   ag_packed_weights** out) {
    if (!B_list || G < 1 || !plan || !amap || !dst || !out || K <= 0 || N <= 0 || (N % G)) return AG_ERR_ARG;
    for (int g = 0; g < G; ++g)
        if (!B_list[g]) return AG_ERR_ARG;
    const int n_src = N / G;
    if (G > 1 && (n_src % 128)) return AG_ERR_ARG;  // experts must start on a page-column boundary
    *out = nullptr;
    const int32_t* h = plan->header;
    if ((h[H_TILE_N] != 128 && h[H_TILE_N] != 256) || h[H_N] != N || h[H_K] != K || (K % SK_BK)) return AG_ERR_ARG;
    if (amap->base != dst || amap->bytes != dst_bytes) return AG_ERR_STALE_AMAP;
    const int tiles_m = h[H_TILES_M], tiles_n = h[H_TILES_N], ksp = h[H_KSPLITS];
    const int ppc = h[H_TILE_N] / 128;          // 128-column blocks per unit column
    const int n_blocks = tiles_n * ppc;
    const int ppt = K / 16;
    const size_t n_pages = (size_t)n_blocks * ppt;
    // die of every unit from the plan's die queues
    const PlanLayout& lay = plan->lay;
    const int32_t* img = plan->h_image.data();
    std::vector<uint8_t> unit_die(lay.n_units, 0);
    for (int e = img[lay.die_q_off() + 1]; e < lay.n_units; ++e) unit_die[img[lay.die_q() + e]] = 1;
    // two logical views over the chunk pairs: page p of view d = the chunk of pair p that sits on die d;
    // a page goes to the view of the die that runs most of the units reading it (tie -> die 0)
    ag_packed_weights* w = new (std::nothrow) ag_packed_weights();
    if (!w) return AG_ERR_NOMEM;
    w->K = K; w->N = N; w->tiles_n = n_blocks; w->pages_per_tile = ppt; w->n_pages = n_pages;
    w->dst = (const uint8_t*)dst; w->dst_bytes = dst_bytes; w->d_page_table = nullptr;
    w->h_page_table.resize(n_pages);
    w->quad_free_bit = -1;
    w->d_quad_base = nullptr;
    const int per = plan->kslabs_per_split;
    auto owner_die = [&](int pc, int k16) {   // the die that runs most of the units reading this page (tie -> die 0)
        const int tn = pc / ppc, ks = (k16 * 16 / SK_BK) / per;
        int votes[2] = {0, 0};
        for (int tm = 0; tm < tiles_m; ++tm) votes[unit_die[((size_t)tm * tiles_n + tn) * ksp + ks]]++;
        return votes[0] >= votes[1] ? 0 : 1;
    };
    // Grouped layout: if the map follows an XOR hash that uses chunk-index bits 0 and 1 and
    // leaves some bit f >= 2 out, the chunks {q, q+a, q+F, q+F+a} (F = 2^f; a = 3 for q = 0 mod 4, a = 1 for
    // q = 1 mod 4; bit f of q clear) always share a die.  The four pages of a k-slab then go to one such group and
    // the kernel fetches them with one strided copy instead of four.
    std::vector<int32_t> quad_base;
    if (!(flags & 1u)) {
        uint32_t mask = 0;
        size_t violations = 0;
        if (ag_affinity_fit_hash(amap, &mask, &violations) == AG_OK && (mask & 3u) == 3u &&
            violations * 50 <= amap->n_chunks) {
            int f = -1;
            for (int b = 2; b < 9 && f < 0; ++b)
                if (!((mask >> b) & 1u)) f = b;
            if (f >= 0) {
                const size_t F = (size_t)1 << f;
                // the hash works on addresses: chunk-index bits are those of (buffer base / 4 KB + q)
                const size_t first = ((uintptr_t)dst / AG_CHUNK_BYTES) % 512;
                std::vector<int32_t> groups[2];
                for (size_t q = 0; q + F + 3 < amap->n_chunks; ++q) {
                    const size_t qa = first + q;
                    if ((qa & F) || (qa & 3) > 1) continue;
                    const size_t a = (qa & 3) == 0 ? 3 : 1;
                    const uint8_t d0 = amap->h_die_of_chunk[q];
                    if (amap->h_die_of_chunk[q + a] == d0 && amap->h_die_of_chunk[q + F] == d0 &&
                        amap->h_die_of_chunk[q + F + a] == d0)
                        groups[d0].push_back((int32_t)q);   // a group whose chunks disagree (noise) is left out
                }
                size_t need[2] = {0, 0};
                for (int pc = 0; pc < n_blocks; ++pc)
                    for (int k16 = 0; k16 < ppt; k16 += 4) need[owner_die(pc, k16)]++;
                if (need[0] <= groups[0].size() && need[1] <= groups[1].size()) {
                    size_t nxt[2] = {0, 0};
                    quad_base.resize(n_pages / 4);
                    for (int pc = 0; pc < n_blocks; ++pc)
                        for (int k16 = 0; k16 < ppt; k16 += 4) {
                            const int d = owner_die(pc, k16);
                            const int32_t q = groups[d][nxt[d]++];
                            const int32_t a = ((first + (size_t)q) & 3) == 0 ? 3 : 1;
                            const size_t p0 = (size_t)pc * ppt + k16;
                            quad_base[p0 / 4] = q | (a == 1 ? (1 << 30) : 0);   // bit 30: group class (a = 1)
                            w->h_page_table[p0] = q;
                            w->h_page_table[p0 + 1] = q + a;
                            w->h_page_table[p0 + 2] = q + (int32_t)F;
                            w->h_page_table[p0 + 3] = q + (int32_t)F + a;
                        }
                    w->quad_free_bit = f;
                }
            }
        }
    }
    if (w->quad_free_bit < 0) {
        // two logical views over the chunk pairs: page p of view d = the chunk of pair p that sits on die d
        size_t next[2] = {0, 0};
        for (int pc = 0; pc < n_blocks; ++pc)
            for (int k16 = 0; k16 < ppt; ++k16) {
                const int d = owner_die(pc, k16);
                const size_t pair = next[d]++;
                if (2 * pair + 1 >= amap->n_chunks) {
                    delete w;
                    return AG_ERR_ARG;  // destination too small for this die's view
                }
                w->h_page_table[(size_t)pc * ppt + k16] =
                    (int32_t)(2 * pair + (amap->h_die_of_chunk[2 * pair] == d ? 0 : 1));
            }
    } else {
        // one box = the four pages of a group: [128 bf16][16 rows][2 x a chunks][2 x F chunks][base chunk]
        EncodeTiledFn enc = get_encode_tiled();
        const cuuint64_t F = (cuuint64_t)1 << w->quad_free_bit;
        for (int cls = 0; cls < 2; ++cls) {
            const cuuint64_t a = cls == 0 ? 3 : 1;
            cuuint64_t dims[5] = {128, 16, 2, 2, (cuuint64_t)amap->n_chunks};
            cuuint64_t strides[4] = {256, a * AG_CHUNK_BYTES, F * AG_CHUNK_BYTES, AG_CHUNK_BYTES};
            cuuint32_t box[5] = {128, 16, 2, 2, 1};
            cuuint32_t estr[5] = {1, 1, 1, 1, 1};
            if (!enc || enc(&w->tm_quad[cls], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, dst, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
                delete w;
                return AG_ERR_CUDA;
            }
        }
    }
    {
        // the packed buffer as a 3-D tensor [chunk][16 rows][128 bf16]: one box of (128, 16, 1) is one page,
        // landing in shared memory in the page's own byte order (no swizzle)
        EncodeTiledFn enc = get_encode_tiled();
        cuuint64_t dims[3] = {128, 16, (cuuint64_t)amap->n_chunks};
        cuuint64_t strides[2] = {256, AG_CHUNK_BYTES};
        cuuint32_t box[3] = {128, 16, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (!enc || enc(&w->tm_pages, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, dst, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            delete w;
            return AG_ERR_CUDA;
        }
    }
    cudaError_t e = cudaMalloc(&w->d_page_table, sizeof(int32_t) * n_pages);
    if (e == cudaSuccess)
        e = cudaMemcpy(w->d_page_table, w->h_page_table.data(), sizeof(int32_t) * n_pages, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && w->quad_free_bit >= 0) {
        e = cudaMalloc(&w->d_quad_base, sizeof(int32_t) * quad_base.size());
        if (e == cudaSuccess)
            e = cudaMemcpy(w->d_quad_base, quad_base.data(), sizeof(int32_t) * quad_base.size(), cudaMemcpyHostToDevice);
    }
    const size_t pages_per_src = n_pages / G;
    for (int g = 0; g < G && e == cudaSuccess; ++g) {
        k_pack_weights<<<(unsigned)pages_per_src, 128>>>((const uint16_t*)B_list[g], K, n_src, ppt,
                                                        w->d_page_table + (size_t)g * pages_per_src, (uint8_t*)dst);
        count_launch();
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        cudaFree(w->d_page_table);
        cudaFree(w->d_quad_base);
        delete w;
        return cuda_fail(e);
    }
    *out = w;
    return AG_OK;
}

extern "C" ag_status ag_pack_weights_ex(const void* const* B_list, int G, int K, int N_expert, const ag_plan* plan,
                                        const ag_affinity_map* amap, void* dst, size_t dst_bytes, uint32_t flags,
                                        ag_packed_weights** out) {
    if (G < 1 || N_expert <= 0 || (long long)G * N_expert > 0x7fffffff) return AG_ERR_ARG;
    return pack_weights_impl(B_list, G, K, G * N_expert, plan, amap, dst, dst_bytes, flags, out);
}

extern "C" ag_status ag_packed_info(const ag_packed_weights* w, int32_t* group_free_bit) {
    if (!w || !group_free_bit) return AG_ERR_ARG;
    *group_free_bit = w->quad_free_bit;
    return AG_OK;
}

extern "C" ag_status ag_pack_weights(const void* B, int K, int N, const ag_plan* plan, const ag_affinity_map* amap,
                                     void* dst, size_t dst_bytes, ag_packed_weights** out) {
    const void* list[1] = {B};
    return pack_weights_impl(list, 1, K, N, plan, amap, dst, dst_bytes, 0, out);
}

extern "C" ag_status ag_pack_weights_grouped(const void* const* B_list, int G, int K, int N_expert, const ag_plan* plan,
                                             const ag_affinity_map* amap, void* dst, size_t dst_bytes,
                                             ag_packed_weights** out) {
    if (G < 1 || N_expert <= 0 || (long long)G * N_expert > 0x7fffffff) return AG_ERR_ARG;
    return pack_weights_impl(B_list, G, K, G * N_expert, plan, amap, dst, dst_bytes, 0, out);
}

// ---- grouped (MoE-shaped) decode GEMM -------------------------------------------------------------------
extern "C" void ag_group_desc_destroy(ag_group_desc* d) {
    if (!d) return;
    cudaFree(d->d_tm_a);
    cudaFree(d->d_tm_w);
    cudaFree(d->d_tm_c);
    cudaFree(d->d_rows);
    cudaFree(d->d_row_off);
    delete d;
}

extern "C" ag_status ag_group_desc_create(const void* A_all, void* C_all, const int32_t* rows, int G,
                                          const void* const* B_list, int N_expert, int K, int tile_m,
                                          ag_group_desc** out) {
    if (!A_all || !C_all || !rows || !out || G < 1 || G > 4096 || N_expert <= 0 || K <= 0) return AG_ERR_ARG;
    const bool dense = tile_m == 256;  // block pairs, 256 x 256 units; else decode-shaped (rows <= tile_m)
    if ((tile_m != 16 && tile_m != 32 && !dense) || (N_expert % (dense ? 256 : SK_BN)) || (K % 8)) return AG_ERR_ARG;
    if (((uintptr_t)A_all | (uintptr_t)C_all) & 15u) return AG_ERR_ARG;
    *out = nullptr;
    long long total = 0;
    for (int g = 0; g < G; ++g) {
        if (rows[g] < 0 || (!dense && rows[g] > tile_m)) return AG_ERR_ARG;
        total += rows[g];
    }
    if (total < 1) return AG_ERR_ARG;
    ag_group_desc* d = new (std::nothrow) ag_group_desc();
    if (!d) return AG_ERR_NOMEM;
    d->G = G; d->N = N_expert; d->K = K; d->tile_m = tile_m; d->total_rows = total;
    d->A_all = A_all; d->C_all = C_all;
    d->d_tm_a = nullptr; d->d_tm_w = nullptr; d->d_tm_c = nullptr; d->d_rows = nullptr; d->d_row_off = nullptr;
    d->w_blocks = (N_expert % 64 == 0) ? 1 : 0;
    d->rows.assign(rows, rows + G);
    d->row_off.resize(G);
    std::vector<CUtensorMap> ha(G), hw(B_list ? G : 0), hc(dense ? G : 0);
    const uint32_t a_box_rows = dense ? 128 : (uint32_t)tile_m;
    long long off = 0;
    for (int g = 0; g < G; ++g) {
        d->row_off[g] = (int)off;
        // an expert without rows still gets a (one-row) view inside the buffer; nothing of it is stored
        const long long first = std::min(off, total - 1);
        const int n_rows = std::max(1, rows[g]);
        const char* base = (const char*)A_all + (size_t)first * K * 2;
        const uint64_t view_rows = (uint64_t)std::min<long long>(n_rows, total - first);
        if (!encode_2d(&ha[g], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, view_rows, K, SK_BK, a_box_rows)) {
            delete d;
            return AG_ERR_CUDA;
        }
        if (dense) {
            float* cbase = (float*)C_all + (size_t)first * N_expert;
            if (!encode_2d(&hc[g], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, cbase, view_rows, N_expert, 32, 32)) {
                delete d;
                return AG_ERR_CUDA;
            }
        }
        if (B_list) {
            if (!B_list[g] || ((uintptr_t)B_list[g] & 15u)) { delete d; return AG_ERR_ARG; }
            const bool ok = d->w_blocks ? encode_b_blocks(&hw[g], B_list[g], K, N_expert, SK_BK, 2)
                                        : encode_2d(&hw[g], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B_list[g], K, N_expert, 64, SK_BK);
            if (!ok) { delete d; return AG_ERR_CUDA; }
        }
        off += rows[g];
    }
    cudaError_t e = cudaMalloc(&d->d_tm_a, sizeof(CUtensorMap) * G);
    if (e == cudaSuccess) e = cudaMemcpy(d->d_tm_a, ha.data(), sizeof(CUtensorMap) * G, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && B_list) {
        e = cudaMalloc(&d->d_tm_w, sizeof(CUtensorMap) * G);
        if (e == cudaSuccess) e = cudaMemcpy(d->d_tm_w, hw.data(), sizeof(CUtensorMap) * G, cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess && dense) {
        e = cudaMalloc(&d->d_tm_c, sizeof(CUtensorMap) * G);
        if (e == cudaSuccess) e = cudaMemcpy(d->d_tm_c, hc.data(), sizeof(CUtensorMap) * G, cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMalloc(&d->d_rows, sizeof(int) * G);
    if (e == cudaSuccess) e = cudaMemcpy(d->d_rows, d->rows.data(), sizeof(int) * G, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&d->d_row_off, sizeof(int) * G);
    if (e == cudaSuccess) e = cudaMemcpy(d->d_row_off, d->row_off.data(), sizeof(int) * G, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        ag_group_desc_destroy(d);
        return cuda_fail(e);
    }
    *out = d;
    return AG_OK;
}

extern "C" ag_status gemm_persistent_grouped(const ag_group_desc* d, const ag_packed_weights* W, const ag_plan* plan,
                                             void* cuda_stream) {
    if (!d || !plan) return AG_ERR_ARG;
    const int32_t* h = plan->header;
    // the plan sees the experts side by side: N = G * N_expert, M = the largest row count of an expert
    if (h[H_N] != d->G * d->N || h[H_K] != d->K || h[H_TILE_M] != d->tile_m) return AG_ERR_ARG;
    for (int g = 0; g < d->G; ++g)
        if (d->rows[g] > h[H_M]) return AG_ERR_ARG;
    if (d->tile_m == 256)  // many rows per expert: block pairs, per-expert A / B / C views
        return gemm_pair_dispatch(d->A_all, nullptr, W, d->C_all, h[H_M], h[H_N], h[H_K], plan,
                                  reinterpret_cast<cudaStream_t>(cuda_stream), d);
    if (h[H_M] > d->tile_m) return AG_ERR_ARG;
    return gemm_skinny_dispatch(d->A_all, nullptr, W, d->C_all, h[H_M], h[H_N], h[H_K], plan, plan->d_partial, plan->d_sem,
                                reinterpret_cast<cudaStream_t>(cuda_stream), d);
}

extern "C" ag_status ag_packed_page_table(const ag_packed_weights* w, int32_t* outp, size_t cap, size_t* n_pages) {
    if (!w) return AG_ERR_ARG;
    if (n_pages) *n_pages = w->n_pages;
    if (!outp) return n_pages ? AG_OK : AG_ERR_ARG;
    if (cap < w->n_pages) return AG_ERR_ARG;
    memcpy(outp, w->h_page_table.data(), w->n_pages * sizeof(int32_t));
    return AG_OK;
}

extern "C" void ag_packed_destroy(ag_packed_weights* w) {
    if (!w) return;
    cudaFree(w->d_quad_base);
    cudaFree(w->d_page_table);
    delete w;
}

extern "C" ag_status gemm_persistent_packed(const void* A, const ag_packed_weights* W, void* Cout, int M, int N, int K,
                                            const ag_plan* plan, void* cuda_stream) {
    if (!A || !W || !Cout || !plan) return AG_ERR_ARG;
    if (plan->header[H_TILE_M] == 256)  // dense plan of block pairs over packed B panels
        return gemm_pair_dispatch(A, nullptr, W, Cout, M, N, K, plan, reinterpret_cast<cudaStream_t>(cuda_stream));
    return gemm_skinny_dispatch(A, nullptr, W, Cout, M, N, K, plan, plan->d_partial, plan->d_sem,
                                reinterpret_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the decode-shaped GEMM.
//
// Some callers must not allocate device memory at the moment they need the GEMM: an inference
// server that has handed every free byte of the GPU to its own arena (cudaMalloc simply fails
// there), a request loop with a latency budget that an allocator call would break, or code
// running between other libraries' strict "no allocation after start-up" phases.  For them the
// split-K workspace lives in the library image itself: a fixed array in device memory that exists
// on every GPU from the moment the library is loaded there until the process ends.
//
// The array's name is only a host-side handle; the address the kernel needs is asked from the
// runtime once per device (cudaGetSymbolAddress, with that device current) and remembered.
constexpr size_t kNoAllocSemBytes = 16 * 1024;                   // 4096 arrival counters = 1024 tiles of 128 columns
constexpr size_t kNoAllocPartialBytes = 8u * 1024 * 1024;        // 2 Mi fp32 partial sums
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocSemBytes + kNoAllocPartialBytes];

namespace {
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[64] = {nullptr};   // device address of g_noalloc_scratch, per device ordinal
}  // namespace

extern "C" ag_status gemm_persistent_noalloc(const void* A, const void* B, void* Cout, int M, int N, int K,
                                             const ag_plan* plan, void* cuda_stream) {
    if (!A || !B || !Cout || !plan) return AG_ERR_ARG;
    const int32_t* h = plan->header;
    if (h[H_TILE_M] > 32) return AG_ERR_ARG;  // only decode-shaped plans use a workspace
    const int ksp = h[H_KSPLITS], tiles_n = h[H_TILES_N];
    // limits of the built-in workspace
    if ((size_t)tiles_n * 4 * sizeof(int) > kNoAllocSemBytes) return AG_ERR_ARG;
    if (ksp > 1 && (size_t)ksp * (size_t)M * (size_t)N * sizeof(float) > kNoAllocPartialBytes) return AG_ERR_ARG;
    int dev = 0;
    AG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return AG_ERR_ARG;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            // first call on this device: resolve the array's device address (not an allocation)
            void* ptr = nullptr;
            AG_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
            g_noalloc_ptr[dev] = ptr;
        }
        scratch = g_noalloc_ptr[dev];
    }
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    int* sem = reinterpret_cast<int*>(scratch);
    float* partial = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + kNoAllocSemBytes);
    // the counters must start at zero; whatever an earlier call left behind is wiped on the same stream
    AG_CUDA(cudaMemsetAsync(sem, 0, (size_t)tiles_n * 4 * sizeof(int), stream));
    return gemm_skinny_dispatch(A, B, nullptr, Cout, M, N, K, plan, partial, sem, stream);
}
