// Decode-shaped (skinny) persistent GEMM: C[M x N] = A[M x K] * B[K x N] with M <= 128.  The
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
// Split-K units either add their sums into a zeroed C with reductions in memory, or write them to a workspace
// whose slices a second kernel (k_reduce_splits) adds in ascending split order (bit-reproducible).
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>

#include "persist.cuh"

namespace ag {

constexpr int SK_BN = 128;     // weight columns per unit
constexpr int SK_BK = 64;      // k-slab
// Two things shape the pipeline (both measured on B200):
//  - a warp gets only about two bulk copies in flight whatever their size (one thread issuing 16 KB copies streams
//    35 GB/s from DRAM with 2, 6 or 12 stages, four warps issuing the same copies 139 GB/s), so the weight copies
//    are issued by SK_WPROD warps in turn and the activation copies by yet another warp;
//  - the thread that issues the MMAs pays a fixed cost per stage (barrier wait, fence, commit) on top of the issue of
//    its MMAs, however small they are: a stage therefore holds two k-slabs (32 KB of weights, 8 MMAs), two warps
//    issue (see the MMA role), and each runs its loop with all 32 lanes and lets one elected lane issue (elect_one in
//    ptx.cuh: 250 ns per stage for the issuing thread instead of 485 ns from a lane-0-only branch).
constexpr int SK_SLABS = 2;    // k-slabs per weight stage
constexpr int SK_WPROD = 3;    // warps that issue weight copies (stage i of the block's run belongs to warp i mod SK_WPROD)
constexpr int SK_STAGES = 6;   // (at most) two stages per issuing warp; even, so that a buffer's parity is the parity of its place in the run
constexpr int SK_NMMA = 2;     // warps that may issue MMAs: thread t owns the stage buffers of parity t (see the MMA role)
// With 64 or 128 activation rows an MMA takes 56-64 cycles and a k-slab of activations 8-16 KB: one MMA-issuing thread
// keeps up, and the activations of a stage's two k-slabs travel with its weights (one stage = 32 KB of weights + 16 or
// 32 KB of activations, filled by the same warp onto the same barrier), so that both have the same pipeline depth.
__host__ __device__ constexpr bool sk_unified(int nm) { return nm >= 64; }
__host__ __device__ constexpr int sk_stages(int nm) { return nm == 64 ? 4 : nm == 128 ? 3 : SK_STAGES; }
__host__ __device__ constexpr int sk_nmma(int nm) { return nm >= 64 ? 1 : SK_NMMA; }
constexpr int SK_THREADS = (2 + kEpiWarps + SK_WPROD + (SK_NMMA - 1)) * 32;   // scheduler, MMA issuer, epilogue warps, weight producers, second MMA issuer
constexpr int SK_MMA2_WARP = 2 + kEpiWarps + SK_WPROD;
constexpr int SK_SLAB_BYTES = SK_BN * SK_BK * 2;   // 16 KB of weights per k-slab
constexpr int SK_W_BYTES = SK_SLABS * SK_SLAB_BYTES;
// Activations come in groups of SK_AGRP k-slabs, one copy per group (A seen as [K/64][M][64]): with one copy
// per k-slab the warp that issues them - two copies in flight, each an L2 round trip - capped the whole
// pipeline at one slab per ~400 ns, the same 42 GB/s per SM that a single weight-issuing thread reaches.
constexpr int SK_ASTAGES = 2;
constexpr int SK_A_STAGE_MAX = 16 * 1024;          // 8 k-slabs of 16 rows, or 4 k-slabs of 32 rows
__host__ __device__ constexpr int sk_agrp(int nm) { return nm >= 64 ? 2 : SK_A_STAGE_MAX / (nm * SK_BK * 2); }   // 64 / 128 rows: 2 k-slabs (16 / 32 KB)
__host__ __device__ constexpr int sk_a_stage_bytes(int nm) { return sk_agrp(nm) * nm * SK_BK * 2; }
__host__ __device__ constexpr int sk_stage_bytes(int nm) { return SK_W_BYTES + (sk_unified(nm) ? sk_a_stage_bytes(nm) : 0); }
__host__ __device__ constexpr int sk_smem_bytes(int nm) {
    return sk_stages(nm) * sk_stage_bytes(nm) + (sk_unified(nm) ? 0 : SK_ASTAGES * sk_a_stage_bytes(nm)) + 1024 + 1024;
}
// The tensor core takes ~45 cycles for an MMA this small whether or not it adds to the accumulator of the one
// before (measured), so one accumulator per unit is enough.

struct SkinnyCtl {
    uint64_t full[SK_STAGES];
    uint64_t empty[SK_STAGES];
    uint64_t a_full[SK_ASTAGES];   // activations of a group of SK_AGRP k-slabs have landed
    uint64_t a_empty[SK_ASTAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t sched_full[kRing];
    uint64_t sched_empty[kRing];
    uint64_t mma_drain[SK_NMMA];
    int ring[kRing];
    uint32_t tmem_base;
    int abort_flag;
    int member;
    int4 quick;
};

struct SkinnyArgs {
    const uint8_t* packed;        // packed weights base (PACKED) or null
    const int32_t* page_table;    // device (PACKED)
    const int32_t* quad_base;     // device (PACKED, grouped layout): first chunk of each k-slab's group, or null
    int consecutive;              // 1 (PACKED): logical page p is chunk p - a stage's pages are one contiguous run, one plain copy
    int quad_f;                   // chunk distance 2^free_bit between the two halves of a group
    int quad_f_bit;               // free_bit
    int pages_per_tile;
    float* C;
    float* partial;               // [k_splits][M][N] or null when k_splits == 1
    // grouped (MoE-shaped) operation: the plan's N is G experts side by side, expert g = column tiles
    // [g * tiles_per_group, (g + 1) * tiles_per_group); null / 0 when there is a single problem
    const CUtensorMap* g_tm_a;    // device [G]: activations of expert g (rows of the stacked A)
    const CUtensorMap* g_tm_w;    // device [G]: row-major weights of expert g (not PACKED)
    const int* g_rows;            // device [G]
    const int* g_row_off;         // device [G]
    int tiles_per_group;
    int n_group;                  // columns of one expert
    int release_next;             // 1: let the next launch on the stream start while this one is still running
    int a_after_prior;            // 1: the activations may be the product of the launch before: read them only after it has completed
    int stages;                   // weight stages in use (at most sk_stages(NM), a multiple of the MMA-issuing threads)
    int producers;                // copying warps in use (at most SK_WPROD)
    // closed form of the page table (PACKED): see table_entry in the kernel
    const int32_t* unit_base;     // device [tiles_n * k_splits] or null (then the tables above are read)
    const uint32_t* page_bits;    // device: one hash bit per 2 MiB page of the packed buffer
    uint32_t hash_mask;
    int hash_first;
    int hash_t0;                  // groups of four chunks that start below hash_first (grouped layout)
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

// a role that gave up lingers this long (bounded) so that copies already in flight land before the block leaves
__device__ __forceinline__ void linger_for_copies() {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
}

template <int NM, bool PACKED>
__global__ void __launch_bounds__(SK_THREADS, 1)
k_gemm_skinny(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
              const __grid_constant__ CUtensorMap tm_w2, const PersistParams p, const SkinnyArgs x) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    constexpr uint32_t kASlab = NM * SK_BK * 2;          // activations of one k-slab
    constexpr int SK_AGRP = sk_agrp(NM);                 // k-slabs per activation copy
    constexpr uint32_t kAStage = SK_AGRP * kASlab;
    constexpr int kStages = sk_stages(NM);               // weight stages
    constexpr int kNMMA = sk_nmma(NM);                   // MMA-issuing threads at work
    constexpr bool kUnified = sk_unified(NM);            // activations inside the weight stages
    constexpr uint32_t kStageBytes = sk_stage_bytes(NM);
    const uint32_t ring_n = (uint32_t)x.stages;          // stages of the ring in use
    const uint32_t a_base = base + kStages * kStageBytes;
    SkinnyCtl* ctl = reinterpret_cast<SkinnyCtl*>(smem + kStages * kStageBytes + (kUnified ? 0 : SK_ASTAGES * kAStage));
    constexpr uint32_t kAccCols = NM;                    // columns of one accumulator
    constexpr uint32_t kTmemCols = 2 * kNMMA * kAccCols < 32 ? 32 : 2 * kNMMA * kAccCols;   // two units in flight, one accumulator per MMA-issuing thread each
    volatile int* abort_flag = &ctl->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int my_sm = (int)smid();
    // overlap_launches: the launch that follows on the stream (this library's, by the caller's promise) may be
    // scheduled as soon as every block of this one has got this far; its blocks move in as SMs become free
    if (x.release_next && tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // One 16-byte entry tells this block its slot, its list and the list's first unit; the claim follows at once.
    if (tid == 0) {
        ctl->abort_flag = 0;
        const int4 qk = p.quick[my_sm];
        ctl->quick = qk;
        ctl->member = qk.x >= 0 && atomicMax(&p.claimed[qk.x], p.epoch) < p.epoch;
    } else if (tid == 64) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < SK_ASTAGES; ++i) {
            mbar_init(smem_u32(&ctl->a_full[i]), 1);
            mbar_init(smem_u32(&ctl->a_empty[i]), kNMMA);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), kNMMA);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), kEpiWarps);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&ctl->sched_full[i]), 1);
            mbar_init(smem_u32(&ctl->sched_empty[i]), kNMMA + kEpiWarps + SK_WPROD);
        }
        for (int i = 0; i < SK_NMMA; ++i) mbar_init(smem_u32(&ctl->mma_drain[i]), 1);
        mbar_fence_init();
        prefetch_tmap(&tm_a);
        if (!PACKED || x.quad_base) prefetch_tmap(&tm_w);
    }
    __syncthreads();
    const int4 quick = ctl->quick;
    const int slot = quick.x;
    if (!ctl->member) {
        if (slot < 0) wait_until_manned(p);
        return;
    }
    const uint64_t limit = p.wait_limit_ns;
    // tensor memory is needed by the MMA issuer and the epilogue only: the copy-issuing warps do not wait for it
    uint32_t tmem_base = 0;
    if ((warp >= 1 && warp < 2 + kEpiWarps) || warp == SK_MMA2_WARP) {
        if (warp == 1) {
            tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
            tmem_relinquish();
        }
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"((SK_NMMA + kEpiWarps) * 32) : "memory");
        tc_fence_after();
        tmem_base = ctl->tmem_base;
    }

    if (warp == 0) {
        // ------------------------------------------------ scheduler + activation copies (lane 0)
        UnitSource src(p, slot, lane, quick.y, quick.z, quick.w);
        uint32_t it = 0, git = 0;
        int ok = 1;
        while (ok) {
            int u;
            if (p.static_assign) {
                u = src.next_listed(lane);
                while (u < 0 && ok) {
                    // Own list done.  Planned SMs that never got a block are looked for only now that the
                    // consumers have taken the last unit off the ring: by then every block of the launch has
                    // long started, and the scan runs while the last unit is being streamed.
                    if (it > 0 && lane == 0 &&
                        !mbar_wait_idle(smem_u32(&ctl->sched_empty[(it - 1) % kRing]), ((it - 1) / kRing) & 1, abort_flag, limit)) {
                        report_timeout(p, 1);
                        ok = 0;
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok || !src.adopt(lane)) break;
                    u = src.next_listed(lane);
                }
            } else {
                u = src.next(lane);
            }
            if (!ok) break;
            if (u >= 0 && x.g_rows) {
                // grouped operation: an expert without rows has nothing to compute - its units are ticked off here and
                // its weights are never read (in a mixture-of-experts layer most experts are idle in most steps)
                const int tn_u = (u / p.k_splits) % p.tiles_n;
                if (x.g_rows[tn_u / x.tiles_per_group] == 0) {
                    if (lane == 0) {
                        p.tile_owner[u] = my_sm;
                        if (p.unit_times) p.unit_times[2 * u] = p.unit_times[2 * u + 1] = globaltimer_ns();
                        atomicAdd(&p.tile_count[u], 1);
                    }
                    continue;
                }
            }
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
            ++it;
            if (!ok || u < 0) break;
            const int ks = u % p.k_splits, tn = (u / p.k_splits) % p.tiles_n;
            const int grp = x.tiles_per_group ? tn / x.tiles_per_group : 0;      // expert of this column tile
            const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
            const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
            if (!kUnified && lane == 0) {
                const CUtensorMap* ma = x.g_tm_a ? &x.g_tm_a[grp] : &tm_a;
                // (this kernel may have started early: the weights stream at once, the activations - which the launch
                // before may have written - only after that launch has completed)
                if (git == 0 && x.a_after_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
                for (int g0 = s0; g0 < s1; g0 += SK_AGRP, ++git) {
                    const int j = git % SK_ASTAGES;
                    if (!mbar_wait_idle(smem_u32(&ctl->a_empty[j]), ((git / SK_ASTAGES) & 1) ^ 1, abort_flag, limit)) {
                        report_timeout(p, 2);
                        ok = 0;
                        break;
                    }
                    const uint32_t bar = smem_u32(&ctl->a_full[j]);
                    const uint32_t dst = a_base + j * kAStage;
                    if (p.a_blocks) {
                        // the whole group with one copy; slabs past the end of K are zero-filled
                        mbar_expect_tx(bar, kAStage);
                        tma_load_3d(dst, ma, bar, 0, 0, g0);
                    } else {
                        const int n = min(SK_AGRP, s1 - g0);
                        mbar_expect_tx(bar, n * kASlab);
                        for (int i = 0; i < n; ++i) tma_load_2d(dst + i * kASlab, ma, bar, (g0 + i) * SK_BK, 0);
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
        }
        if (!ok && lane == 0) linger_for_copies();
    } else if (warp >= 2 + kEpiWarps && warp < SK_MMA2_WARP) {
        // ------------------------------------------------ weight copies: warp pw issues k-iterations pw, pw + SK_WPROD, ...
        // For packed weights all 32 lanes fetch the page-table entries of the next eight k-slabs with one load
        // each, so the issuing lane never waits on a table lookup.
        const int pw = warp - (2 + kEpiWarps);
        // Copying warps: their number divides the ring (or the one MMA-issuing thread hands the stages back in order), so
        // that a warp waiting for a stage to come free is never more than one use of that stage ahead of its barrier.
        const int n_prod = x.producers;
        const uint64_t stream_policy = l2_policy_evict_first();  // weights are read once: do not keep them in L2
        uint32_t q0 = 0;      // stage count (over the whole run of this block) before the current unit
        bool a_ready = false; // (activations inside the stages) everything launched before is known to be complete
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
            const int ks = u % p.k_splits, tn = (u / p.k_splits) % p.tiles_n;
            const int grp = x.tiles_per_group ? tn / x.tiles_per_group : 0;      // expert of this column tile
            const int tl = x.tiles_per_group ? tn - grp * x.tiles_per_group : tn;  // tile inside the expert
            const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
            const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
            const int n_st = (s1 - s0 + SK_SLABS - 1) / SK_SLABS;    // stages of this unit: slabs s0 + 2i, s0 + 2i + 1
            // this warp's stages of the unit: i0, i0 + n_prod, ... (a warp beyond the copying ones takes the unit off the ring and copies nothing)
            const int i0 = pw < n_prod ? (pw + n_prod - (int)(q0 % (uint32_t)n_prod)) % n_prod : n_st;
            uint32_t st = (q0 + i0) % ring_n, ph = (((q0 + i0) / ring_n) & 1) ^ 1;   // stage, parity of "stage is free"
            const CUtensorMap* mw = x.g_tm_w ? &x.g_tm_w[grp] : &tm_w;
            // packed weights: lane l < 2 (groups of four pages) or l < 8 (single pages) looks up the chunk of the
            // l-th 16 KB / 4 KB piece of a stage, one stage ahead of the copies
            // Closed form (Eq. 1 of the remapping appendix): the unit's pages are consecutive in the view of its die, so the
            // chunk of a page follows from the unit's first position, the fitted hash mask and one bit per 2 MiB page;
            // one table word per unit instead of one per page or group.
            int ubase = 0;
            if (PACKED && x.unit_base) ubase = x.unit_base[(size_t)tn * p.k_splits + ks];
            auto table_entry = [&](int i) -> int {
                if (!PACKED || i >= n_st || x.consecutive) return 0;
                const int s = s0 + i * SK_SLABS;
                if (x.unit_base) {
                    const int d = (ubase >> 31) & 1, pos0 = ubase & 0x7fffffff;
                    if (x.quad_base) {
                        if (lane >= SK_SLABS || s + lane >= s1) return 0;
                        const int f = x.quad_f_bit;
                        const uint32_t T = (uint32_t)(pos0 + (s - s0) + lane + x.hash_t0);       // run of four chunks that holds the group
                        const uint32_t qa0 = ((T >> (f - 2)) << (f + 1)) | ((T & ((1u << (f - 2)) - 1u)) << 2);
                        const uint32_t cb = (x.page_bits[qa0 >> 14] >> ((qa0 >> 9) & 31)) & 1u;
                        const uint32_t e = (__popc(qa0 & x.hash_mask) & 1u) ^ cb ^ (uint32_t)d;
                        return (int)((qa0 + e - (uint32_t)x.hash_first) | (e << 30));           // bit 30: class of the group (a = 1)
                    }
                    if (lane >= 4 * SK_SLABS || s + (lane >> 2) >= s1) return 0;
                    const uint32_t j = (uint32_t)(pos0 + (s - s0) * 4 + lane);                 // pair of chunks that holds the page
                    const uint32_t qa = (uint32_t)x.hash_first + 2u * j;
                    const uint32_t cb = (x.page_bits[qa >> 14] >> ((qa >> 9) & 31)) & 1u;
                    return (int)(2u * j + ((__popc(qa & x.hash_mask) & 1u) ^ cb ^ (uint32_t)d));
                }
                if (x.quad_base) return (lane < SK_SLABS && s + lane < s1) ? x.quad_base[(size_t)tn * (x.pages_per_tile / 4) + s + lane] : 0;
                return (lane < 4 * SK_SLABS && s + (lane >> 2) < s1) ? x.page_table[(size_t)tn * x.pages_per_tile + (size_t)s * 4 + lane] : 0;
            };
            int next_entry = table_entry(i0);
            for (int i = i0; i < n_st && ok; i += n_prod) {
                const int entry = next_entry;
                next_entry = table_entry(i + n_prod);
                const int s = s0 + i * SK_SLABS;
                const int ns = min(SK_SLABS, s1 - s);
                const uint32_t bar = smem_u32(&ctl->full[st]);
                const uint32_t sw = base + st * kStageBytes;
                if (lane == 0) {
                    if (!mbar_wait(smem_u32(&ctl->empty[st]), ph, abort_flag, limit)) {
                        report_timeout(p, 2);
                        ok = 0;
                    } else {
                        // row-major weights: one box of 128 k rows whatever ns is (rows past K arrive as zeros)
                        uint32_t bytes = PACKED ? ns * SK_SLAB_BYTES : SK_W_BYTES;
                        if (kUnified) bytes += p.a_blocks ? kAStage : ns * kASlab;
                        mbar_expect_tx(bar, bytes);
                        if (kUnified) {
                            // the activations of the stage's k-slabs, behind its weights (when this kernel may have started
                            // early: only once the launch before, which may have written them, has completed)
                            if (!a_ready) {
                                if (x.a_after_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
                                a_ready = true;
                            }
                            const CUtensorMap* ma = x.g_tm_a ? &x.g_tm_a[grp] : &tm_a;
                            if (p.a_blocks) tma_load_3d(sw + SK_W_BYTES, ma, bar, 0, 0, s);
                            else for (int j = 0; j < ns; ++j) tma_load_2d(sw + SK_W_BYTES + j * kASlab, ma, bar, (s + j) * SK_BK, 0);
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (PACKED && x.consecutive) {
                    // pages in consecutive chunks: the stage's two k-slabs are 32 KB in one piece, one plain copy
                    if (lane == 0)
                        bulk_load_hint(sw, x.packed + ((size_t)tn * x.pages_per_tile + (size_t)s * 4) * AG_CHUNK_BYTES,
                                       (uint32_t)(ns * SK_SLAB_BYTES), bar, stream_policy);
                } else if (PACKED && x.quad_base) {
                    // grouped layout: a slab's four pages sit in chunks q, q+a, q+F, q+F+a of one die (a = 3 or 1 by
                    // q mod 4): one strided box brings its 16 KB; bit 30 of the entry = class of the group
                    if (lane < ns)
                        tma_load_5d_hint(sw + lane * SK_SLAB_BYTES, (entry >> 30) ? &tm_w2 : &tm_w, bar, 0, 0, 0, 0,
                                         entry & 0x3fffffff, stream_policy);
                } else if (PACKED) {
                    // one lane per 4 KB page, all in one instruction
                    if (lane < 4 * ns)
                        bulk_load_hint(sw + lane * 4096, x.packed + (size_t)entry * AG_CHUNK_BYTES, 4096, bar, stream_policy);
                } else if (lane == 0) {
                    if (p.b_blocks) {
                        // both 64-column blocks with one copy (B seen as [N/64][K][64])
                        tma_load_3d_hint(sw, mw, bar, 0, s * SK_BK, tl * 2, stream_policy);
                    } else {
                        tma_load_2d_hint(sw, mw, bar, tl * SK_BN, s * SK_BK, stream_policy);
                        tma_load_2d_hint(sw + SK_W_BYTES / 2, mw, bar, tl * SK_BN + 64, s * SK_BK, stream_policy);
                    }
                }
                // this warp's next stage is n_prod stages on
                st += (uint32_t)n_prod;
                if (st >= ring_n) { st -= ring_n; ph ^= 1; }
            }
            q0 += (uint32_t)n_st;
        }
        if (!ok && lane == 0) linger_for_copies();
    } else if (warp == 1 || warp == SK_MMA2_WARP) {
        if (warp == 1 || kNMMA == 2) {
            // ------------------------------------------------ MMA issuers (with 64 or 128 activation rows: warp 1 alone).  Thread t (0: warp 1, 1: the last warp) owns the
            // stage buffers of parity t, i.e. every second stage of the block's run.  One issuing warp feeds 67 GB/s per SM
            // (250 ns per 32 KB stage for eight MMAs, a barrier wait, a fence and a commit), two feed the 120 GB/s that
            // the copy ring delivers.
            // Ownership by buffer, not by position in the unit: a parity wait on a stage barrier is only right for the
            // thread that consumed the buffer's previous contents (a thread a whole lap ahead would see the parity of the
            // lap before as "full").  Inside a unit the thread therefore has the stages of one parity a, and adds them up
            // in accumulator a: accumulator 0 always holds the unit's even stages and accumulator 1 the odd ones, so the
            // value of C does not depend on what the SM ran before.
            // All 32 lanes of the warp run the loop converged; one elected lane issues the MMAs and commits (see elect_one).
            const int t = warp == 1 ? 0 : 1;
            constexpr uint32_t idesc = make_idesc_bf16(128, NM, PACKED ? 0 : 1, 0);
            // descriptors without their start address.  Weights: packed page = no swizzle, 16-byte k chunks 128 B
            // apart (LBO), 8-row groups 256 B apart (SBO); row-major = MN-major with 128-byte swizzle, the two
            // 64-column blocks of a stage half a stage apart (LBO), 8 k rows 1 KB apart (SBO).  The address field
            // counts 16-byte units; shared memory is below 256 KB, so adding to the low word never carries out of it.
            const uint64_t dw_t = PACKED ? make_smem_desc(0, 128, 256, 0) : make_smem_desc(0, SK_W_BYTES / 2, 1024, 2);
            const uint64_t da_t = make_smem_desc(0, 16, 1024, 2);
            constexpr uint32_t kWStep = (PACKED ? 4096u : 2048u) >> 4;   // one K = 16 step inside a weight stage
            constexpr uint32_t kAStepK = 32u >> 4;                       // ... inside an activation slab
            constexpr int kGrpStages = SK_AGRP / SK_SLABS;               // stages per activation buffer (even)
            static_assert(kGrpStages % kNMMA == 0, "every full activation group has stages of both threads");
            static_assert(kStages % kNMMA == 0, "a stage buffer always belongs to the same thread");
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            uint32_t q0 = 0;                          // stages of the units before this one (over the whole run of the block)
            uint32_t git = 0;                         // activation groups before this unit
            uint32_t tile_it = 0;
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
                const int ks = u % p.k_splits;
                const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
                const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
                const int n_slabs = s1 - s0;
                const int n_st = (n_slabs + SK_SLABS - 1) / SK_SLABS;
                const int n_grp = (n_slabs + SK_AGRP - 1) / SK_AGRP;
                const uint32_t acc = tile_it & 1;
                if (!mbar_wait_all(smem_u32(&ctl->tmem_empty[acc]), ((tile_it >> 1) & 1) ^ 1, abort_flag, limit)) {
                    if (lane == 0) report_timeout(p, 4);
                    break;
                }
                tc_fence_after();
                const int a = kNMMA == 2 ? (t - (int)(q0 & 1u)) & 1 : 0;   // parity, inside the unit, of the stages in this thread's buffers
                const uint32_t d_tmem = tmem_base + (acc * kNMMA + a) * kAccCols;
                uint32_t st = (q0 + a) % ring_n, ph = ((q0 + a) / ring_n) & 1;   // this thread's first stage of the unit
                bool first = true;
                if constexpr (kUnified) {
                    // activations behind the weights of the same stage: one barrier per stage, no activation buffers
                    for (int i = 0; i < n_st; ++i) {
                        if (!mbar_wait_all(full0 + st * 8, ph, abort_flag, limit)) {
                            if (lane == 0) report_timeout(p, 5);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t sbase = base + st * kStageBytes;
                        const uint64_t dw = dw_t | (uint64_t)(sbase >> 4);
                        const uint64_t da = da_t | (uint64_t)((sbase + SK_W_BYTES) >> 4);
                        const bool two = n_slabs - i * SK_SLABS > 1;
                        if (elect_one()) {
                            tc_mma_f16(d_tmem, dw, da, idesc, first ? 0u : 1u);
#pragma unroll
                            for (int k4 = 1; k4 < SK_BK / 16; ++k4) tc_mma_f16(d_tmem, dw + k4 * kWStep, da + k4 * kAStepK, idesc, 1u);
                            if (two) {
                                const uint64_t da2 = da + (kASlab >> 4);
#pragma unroll
                                for (int k4 = 0; k4 < SK_BK / 16; ++k4)
                                    tc_mma_f16(d_tmem, dw + (4 + k4) * kWStep, da2 + k4 * kAStepK, idesc, 1u);
                            }
                            tc_commit(empty0 + st * 8);
                        }
                        __syncwarp();
                        first = false;
                        if (++st == ring_n) { st = 0; ph ^= 1; }
                    }
                } else
                for (int g = 0; g < n_grp && ok; ++g) {
                    const uint32_t gi = git + g, aj = gi % SK_ASTAGES, aph = (gi / SK_ASTAGES) & 1;
                    const int i_end = min(n_st, (g + 1) * kGrpStages);
                    int i = g * kGrpStages + a;
                    // (waited for even when nothing of the group is this thread's: its release below must not be
                    // counted among the releases of the group that used the buffer before)
                    if (!mbar_wait_all(smem_u32(&ctl->a_full[aj]), aph, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 9);
                        ok = false;
                        break;
                    }
                    if (i >= i_end) {
                        // a last group of one stage: nothing of it is this thread's
                        if (lane == 0) mbar_arrive(smem_u32(&ctl->a_empty[aj]));
                        break;
                    }
                    uint64_t da = (da_t | (uint64_t)((a_base + aj * kAStage) >> 4)) + (uint32_t)a * (SK_SLABS * (kASlab >> 4));
                    for (; i < i_end; i += kNMMA) {
                        if (!mbar_wait_all(full0 + st * 8, ph, abort_flag, limit)) {
                            if (lane == 0) report_timeout(p, 5);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t dw = dw_t | (uint64_t)((base + st * kStageBytes) >> 4);
                        // the first k-slab of the stage, then the second one if the unit has it
                        const bool two = n_slabs - i * SK_SLABS > 1;
                        if (elect_one()) {
                            tc_mma_f16(d_tmem, dw, da, idesc, first ? 0u : 1u);
#pragma unroll
                            for (int k4 = 1; k4 < SK_BK / 16; ++k4) tc_mma_f16(d_tmem, dw + k4 * kWStep, da + k4 * kAStepK, idesc, 1u);
                            if (two) {
                                const uint64_t da2 = da + (kASlab >> 4);
#pragma unroll
                                for (int k4 = 0; k4 < SK_BK / 16; ++k4)
                                    tc_mma_f16(d_tmem, dw + (4 + k4) * kWStep, da2 + k4 * kAStepK, idesc, 1u);
                            }
                            tc_commit(empty0 + st * 8);
                        }
                        __syncwarp();
                        first = false;
                        st += kNMMA;
                        if (st >= ring_n) { st -= ring_n; ph ^= 1; }
                        da += kNMMA * SK_SLABS * (kASlab >> 4);
                    }
                    if (ok && elect_one()) tc_commit(smem_u32(&ctl->a_empty[aj]));    // this thread's last read of the buffer has been issued
                    __syncwarp();
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->tmem_full[acc]));
                __syncwarp();
                q0 += (uint32_t)n_st;
                git += (uint32_t)n_grp;
                ++tile_it;
            }
            __syncwarp();
            if (*abort_flag) {
                if (elect_one()) {
                    tc_commit(smem_u32(&ctl->mma_drain[t]));
                    int dummy = 0;
                    mbar_wait(smem_u32(&ctl->mma_drain[t]), 0, &dummy, 2000000ull);
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------ epilogue: lane = weight column n, registers = rows m
        // Each epilogue warp owns 32 columns of a tile.  Split-K: either every unit adds its sums to C with reductions
        // in memory (C zeroed beforehand), or it stores them to its split's slice of the workspace and the kernel
        // launched behind this one (k_reduce_splits) adds the slices in ascending split order.
        const int q = warp & 3;
        uint32_t tile_it = 0;
        bool prior_done = false;     // everything launched before this kernel is known to be complete
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
            const int ks = u % p.k_splits, tn = (u / p.k_splits) % p.tiles_n;
            const uint32_t acc = tile_it & 1;
            if (!mbar_wait_warp(smem_u32(&ctl->tmem_full[acc]), (tile_it >> 1) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 7);
                break;
            }
            tc_fence_after();
            // This kernel may have started while the one before it (the zeroing of C, the adding-up of the previous
            // call's workspace, or with overlap_launches the previous GEMM) was still running (programmatic dependent
            // launch): before the first byte is written, make sure that everything before it on the stream has completed.
            if (!prior_done) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                prior_done = true;
            }
            const int n = tn * SK_BN + q * 32 + lane;     // column in the plan's (possibly grouped) N
            const OutView ov = out_view(p, x, tn);
            const int nl = ov.col0 + q * 32 + lane;       // column inside the tile's problem
            const int s0e = min(p.kslabs_total, ks * p.kslabs_per_split), s1e = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
            const bool two = kNMMA == 2 && s1e - s0e > SK_SLABS;   // the unit has stages of the second MMA-issuing thread too
            constexpr int kChunk = NM < 32 ? NM : 32;     // activation rows handled at a time
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kNMMA * kAccCols;
#pragma unroll
            for (int c0 = 0; c0 < NM; c0 += kChunk) {
                float sum[kChunk];
                {
                    // the accumulator of the thread that took the even stages, plus the other one's if the unit has a second stage
                    uint32_t v[kChunk], w[kChunk];
                    if constexpr (kChunk == 16) tmem_ld_32x16(taddr + c0, v); else tmem_ld_32x32(taddr + c0, v);
                    if (two) {
                        if constexpr (kChunk == 16) tmem_ld_32x16(taddr + kAccCols + c0, w); else tmem_ld_32x32(taddr + kAccCols + c0, w);
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int m = 0; m < kChunk; ++m) sum[m] = two ? __uint_as_float(v[m]) + __uint_as_float(w[m]) : __uint_as_float(v[m]);
                }
                if (c0 + kChunk >= NM) {                  // the last chunk has been read: the accumulators may be reused
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
                }
                if (p.k_splits > 1 && x.partial == nullptr) {
                    // in-memory reduction: L2 carries out the additions; nothing comes back, so nothing is waited for
                    if (nl < ov.n_cols) {
#pragma unroll
                        for (int m = 0; m < kChunk; ++m)
                            if (c0 + m < ov.rows) atomicAdd(ov.base + (size_t)(c0 + m) * ov.ld + nl, sum[m]);
                    }
                } else if (p.k_splits > 1) {
                    float* out = x.partial + (size_t)ks * p.M * p.N;   // workspace rows: the plan's M bound, columns: the plan's N
                    if (n < p.N) {
#pragma unroll
                        for (int m = 0; m < kChunk; ++m)
                            if (c0 + m < p.M) out[(size_t)(c0 + m) * p.N + n] = sum[m];
                    }
                } else if (nl < ov.n_cols) {
#pragma unroll
                    for (int m = 0; m < kChunk; ++m)
                        if (c0 + m < ov.rows) ov.base[(size_t)(c0 + m) * ov.ld + nl] = sum[m];
                }
            }
            ++tile_it;
            if (lane == 0 && q == 0) {
                p.tile_owner[u] = my_sm;
                if (p.unit_times) p.unit_times[2 * u + 1] = globaltimer_ns();
                atomicAdd(&p.tile_count[u], 1);
            }
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
    // with overlap_launches this kernel itself may have started early: the GEMM before it may still be adding to C
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x)
        p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Adds the k_splits slices of the workspace in ascending split order and writes C (the bit-reproducible split-K
// mode).  One thread per four consecutive columns of one row; the k_splits loads of a thread are in flight together.
// Launched behind the GEMM with programmatic stream serialization: its blocks may become resident while the GEMM
// runs, release the launch behind them at once and wait for the GEMM's completion before the first load.
__global__ void __launch_bounds__(256) k_reduce_splits(const PersistParams p, const SkinnyArgs x) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int quads_per_row = (p.N + 3) / 4;
    const long long total = (long long)p.M * quads_per_row;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int m = (int)(i / quads_per_row), n = (int)(i % quads_per_row) * 4;
        const int tn = n / SK_BN;
        const OutView ov = out_view(p, x, tn);
        const int nl = ov.col0 + (n - tn * SK_BN);
        if (m >= ov.rows || nl >= ov.n_cols) continue;
        float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k0 = 0; k0 < p.k_splits; k0 += 8) {
            float4 t[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k0 + k < p.k_splits) t[k] = __ldcg(reinterpret_cast<const float4*>(x.partial + ((size_t)(k0 + k) * p.M + m) * p.N + n));
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k0 + k < p.k_splits) { acc4.x += t[k].x; acc4.y += t[k].y; acc4.z += t[k].z; acc4.w += t[k].w; }
        }
        *reinterpret_cast<float4*>(ov.base + (size_t)m * ov.ld + nl) = acc4;
    }
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
                               const PersistParams& gp, const SkinnyArgs& x, cudaStream_t stream, bool may_start_early) {
    static std::atomic<unsigned long long> attr_done{0};
    const cudaError_t attr_err = once_per_device(attr_done, [] {
        return cudaFuncSetAttribute(k_gemm_skinny<NM, PACKED>, cudaFuncAttributeMaxDynamicSharedMemorySize, sk_smem_bytes(NM));
    });
    if (attr_err != cudaSuccess) return launch_failed(plan, attr_err);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(plan->grid_blocks > 0 ? plan->grid_blocks : plan->lay.n_sm);
    cfg.blockDim = dim3(SK_THREADS);
    cfg.dynamicSmemBytes = sk_smem_bytes(NM);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = may_start_early ? 1 : 0;   // may start while the kernel before it (zeroing, previous GEMM) is still running
    const cudaError_t le = cudaLaunchKernelEx(&cfg, k_gemm_skinny<NM, PACKED>, tm_a, tm_w, tm_w2, gp, x);
    if (le != cudaSuccess) return launch_failed(plan, le);
    count_launch();
    return AG_OK;
}

// Shared host path of the two skinny entry points.
ag_status gemm_skinny_dispatch(const void* A, const void* B_rowmajor, const ag_packed_weights* W, void* Cout, int M,
                               int N, int K, const ag_plan* plan, float* partial, cudaStream_t stream,
                               const ag_group_desc* grp) {
    const int32_t* h = plan->header;
    if (M != h[H_M] || N != h[H_N] || K != h[H_K]) return AG_ERR_ARG;
    const int tile_m = h[H_TILE_M];
    if (h[H_TILE_N] != SK_BN || (tile_m != 16 && tile_m != 32 && tile_m != 64 && tile_m != 128) || M > tile_m) return AG_ERR_ARG;
    if (plan->policy.k_unit != SK_BK || (K % 8) || (N % 8)) return AG_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)Cout) & 15u) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    if ((st = refuse_capture(stream)) != AG_OK) return st;
    if ((st = renew_epochs_if_needed(plan, stream)) != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (n_sm != plan->lay.n_sm) return AG_ERR_ARG;
    const int NM = h[H_TILE_M];
    CUtensorMap tm_a, tm_w, tm_w2;
    memset(&tm_w, 0, sizeof tm_w);
    memset(&tm_w2, 0, sizeof tm_w2);
    memset(&tm_a, 0, sizeof tm_a);
    const bool a_blocks = grp ? grp->a_blocks != 0 : (K % SK_BK == 0);
    if (!grp && !(a_blocks ? encode_a_slabs(&tm_a, A, M, K, NM, sk_agrp(NM))
                           : encode_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, M, K, SK_BK, NM)))
        return AG_ERR_CUDA;
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
    if (W) {
        if (W->K != K || W->N != N || (K % SK_BK) || W->tiles_n != h[H_TILES_N]) return AG_ERR_ARG;
        x.packed = W->dst;
        x.page_table = W->d_page_table;
        x.consecutive = W->consecutive;
        x.pages_per_tile = W->pages_per_tile;
        if (W->closed_form && W->k_splits == h[H_KSPLITS]) {   // same units as the packing: positions are per unit
            x.unit_base = W->d_unit_base;
            x.page_bits = W->d_page_bits;
            x.hash_mask = W->hash_mask;
            x.hash_first = W->hash_first;
            x.hash_t0 = W->hash_t0;
        }
        if (W->quad_free_bit >= 0) {
            x.quad_base = W->d_quad_base;
            x.quad_f = 1 << W->quad_free_bit;
            x.quad_f_bit = W->quad_free_bit;
            tm_w = W->tm_quad[0];
            tm_w2 = W->tm_quad[1];
        }
    } else if (grp) {
        if (!grp->d_tm_w) return AG_ERR_ARG;  // the descriptor was made without row-major weights
    } else {
        if (!B_rowmajor || ((uintptr_t)B_rowmajor & 15u)) return AG_ERR_ARG;
        if (N % 64 == 0) {
            if (!encode_b_blocks(&tm_w, B_rowmajor, K, N, SK_SLABS * SK_BK, 2)) return AG_ERR_CUDA;
        } else if (!encode_2d(&tm_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B_rowmajor, K, N, 64, SK_SLABS * SK_BK)) {
            return AG_ERR_CUDA;
        }
    }
    // every argument check has passed: from here on work is queued on the stream
    const bool zeroing = h[H_KSPLITS] > 1 && !x.partial;
    // Overlapping launches: the blocks of the next launch find room where a block of this one has left, one per SM, and
    // no block of the launch after next can start before every block of the next one has started.  With a plan for part
    // of the chip the next launch's first blocks land on the unplanned SMs while this launch still holds the planned
    // ones; they stay there until the planned SMs have their blocks (wait_until_manned without its 40 us limit), so that
    // the remaining blocks can only land where this launch's blocks leave.  Static lists only: the queue heads of
    // dynamic plans belong to one launch at a time.
    const bool overlap = plan->policy.overlap_launches && h[H_STATIC] && plan->grid_blocks == 0;
    x.release_next = overlap ? 1 : 0;
    x.a_after_prior = (overlap && plan->policy.overlap_launches != 2) ? 1 : 0;
    x.stages = ring_stages_for(plan, sk_stages(NM), std::min(sk_stages(NM), 2), sk_nmma(NM) == 2, false);
    // Units of at most four stages (128 KB of weights, e.g. N = K = 8192 in 16 k-splits) of row-major weights or of pages in
    // consecutive chunks: a ring of four stages streams 5-6 % more than one of six on the full chip (6.13-6.20 against 5.79-5.83 TB/s) and the same on 37 and 74 SMs; with longer
    // units the deeper ring wins (4 k-splits: 6.81-6.84 against 6.63-6.64 TB/s).
    // Die-local pages are the exception (16 k-splits: 6.11-6.14 TB/s with six stages against 5.88-5.94 with four).
    if (plan->policy.ring_stages <= 0 && sk_stages(NM) == SK_STAGES && (plan->kslabs_per_split + SK_SLABS - 1) / SK_SLABS <= 4 &&
        (!W || W->consecutive))
        x.stages = 4;
    x.producers = x.stages % 3 == 0 ? 3 : x.stages % 2 == 0 ? 2 : sk_nmma(NM) == 1 ? std::min(3, x.stages) : 1;
    if (zeroing) {  // in-memory reduction mode: the adds need a zeroed C (N % 8 == 0 and 16-byte alignment: whole float4s)
        const size_t c_elems = grp ? (size_t)grp->total_rows * (size_t)grp->N : (size_t)M * (size_t)N;
        const size_t n_vec = c_elems / 4;
        const unsigned blocks = (unsigned)std::min<size_t>(148, (n_vec + 255) / 256);
        cudaLaunchConfig_t zc;
        memset(&zc, 0, sizeof zc);
        zc.gridDim = dim3(blocks);
        zc.blockDim = dim3(256);
        zc.stream = stream;
        cudaLaunchAttribute za[1];
        za[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        za[0].val.programmaticStreamSerializationAllowed = 1;
        zc.attrs = za;
        zc.numAttrs = overlap ? 1 : 0;     // may be scheduled while the GEMM before it is finishing; it waits before it writes
        AG_CUDA(cudaLaunchKernelEx(&zc, k_zero_f32, (float4*)Cout, n_vec));
        count_launch();
    }
    PersistParams gp = make_persist_params(plan, M, N, K);
    if (overlap && plan->lay.b < plan->lay.n_sm) gp.manned_wait_ns = gp.wait_limit_ns;
    gp.b_blocks = grp ? ((!W && grp->w_blocks) ? 1 : 0) : ((!W && N % 64 == 0) ? 1 : 0);
    gp.a_blocks = a_blocks ? 1 : 0;
    ag_status ls;
    const bool early = zeroing || overlap;
    if (NM == 16) ls = W ? launch_skinny<16, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early)
                         : launch_skinny<16, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early);
    else if (NM == 32) ls = W ? launch_skinny<32, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early)
                              : launch_skinny<32, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early);
    else if (NM == 64) ls = W ? launch_skinny<64, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early)
                              : launch_skinny<64, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early);
    else ls = W ? launch_skinny<128, true>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early)
                : launch_skinny<128, false>(plan, tm_a, tm_w, tm_w2, gp, x, stream, early);
    if (ls != AG_OK || !x.partial) return ls;
    // bit-reproducible split-K: the workspace slices are added in ascending split order by a second kernel, which may
    // become resident while the GEMM runs and waits for its completion on the device
    const long long quads = (long long)M * ((N + 3) / 4);
    cudaLaunchConfig_t rc;
    memset(&rc, 0, sizeof rc);
    rc.gridDim = dim3((unsigned)std::min<long long>(4 * 148, (quads + 255) / 256));
    rc.blockDim = dim3(256);
    rc.stream = stream;
    cudaLaunchAttribute ra[1];
    ra[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    ra[0].val.programmaticStreamSerializationAllowed = 1;
    rc.attrs = ra;
    rc.numAttrs = 1;
    AG_CUDA(cudaLaunchKernelEx(&rc, k_reduce_splits, gp, x));
    count_launch();
    return AG_OK;
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
    w->consecutive = (flags & 4u) ? 1 : 0;
    w->closed_form = 0; w->k_splits = ksp; w->hash_mask = 0; w->hash_first = 0; w->d_unit_base = nullptr; w->d_page_bits = nullptr;
    w->table_bytes = w->closed_bytes = 0;
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
    if (!(flags & 1u) && !w->consecutive) {
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
    if (w->consecutive) {
        // the placement that ignores the dies: logical page p in chunk p, wherever the hardware's interleaving puts it
        if (n_pages > amap->n_chunks) {
            delete w;
            return AG_ERR_ARG;
        }
        for (size_t i = 0; i < n_pages; ++i) w->h_page_table[i] = (int32_t)i;
    } else if (w->quad_free_bit < 0) {
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
    // Closed form of the tables (Eq. 1 of the remapping appendix).  The measured map must be an exact XOR hash over the
    // chunks in use: mask from ag_affinity_fit_hash, one bit per 2 MiB page by majority, no chunk out of line; the
    // buffer must start on a multiple of four chunks inside its 2 MiB page; decode-shaped plans only (one unit = one
    // run of pages of one die).  Every table entry is then recomputed from the formula and compared; on any
    // difference the tables stay in use.
    if (e == cudaSuccess && !(flags & 2u) && !w->consecutive && tiles_m == 1 && ppc == 1) {
        uint32_t mask = 0;
        const size_t first = ((uintptr_t)dst / AG_CHUNK_BYTES) % 512;
        const int f = w->quad_free_bit;
        bool ok = ag_affinity_fit_hash(amap, &mask, nullptr) == AG_OK && (mask & 1u) && (first % 4) == 0;
        if (ok && f >= 0) ok = (mask & 3u) == 3u && !((mask >> f) & 1u);
        size_t max_chunk = 0;
        for (size_t i = 0; i < n_pages; ++i) max_chunk = std::max(max_chunk, (size_t)w->h_page_table[i]);
        const size_t used = std::min(amap->n_chunks, max_chunk + 1 + (f >= 0 ? ((size_t)1 << f) + 4 : 2));
        std::vector<uint32_t> bits((((first + used) >> 9) + 32) / 32, 0u);
        if (ok) {
            const size_t n2m = ((first + used) >> 9) + 1;
            std::vector<int> ones(n2m, 0), cnt(n2m, 0);
            for (size_t q = 0; q < used; ++q) {
                const size_t qa = first + q;
                ones[qa >> 9] += amap->h_die_of_chunk[q] ^ (__builtin_popcount((uint32_t)qa & mask) & 1);
                cnt[qa >> 9]++;
            }
            for (size_t pg = 0; pg < n2m; ++pg)
                if (2 * ones[pg] > cnt[pg]) bits[pg >> 5] |= 1u << (pg & 31);
        }
        auto page_bit = [&](size_t qa) { return (bits[qa >> 14] >> ((qa >> 9) & 31)) & 1u; };
        std::vector<int32_t> unit_base((size_t)n_blocks * ksp, 0);
        int t0 = 0;
        if (ok && f >= 0) {
            const size_t F = (size_t)1 << f;
            t0 = (int)((first / (2 * F)) * (F / 4) + std::min(first % (2 * F), F) / 4);
        }
        if (ok) {
            // position of every unit's first page in its die's view = pages (or groups) of that die before it
            size_t nxt[2] = {0, 0};
            const int step = f >= 0 ? 4 : 1;                 // pages per position
            for (int pc = 0; pc < n_blocks && ok; ++pc)
                for (int ks = 0; ks < ksp && ok; ++ks) {
                    const int k16_0 = ks * per * 4, k16_1 = std::min(ppt, (ks + 1) * per * 4);
                    const int d = owner_die(pc, k16_0);
                    unit_base[(size_t)pc * ksp + ks] = (int32_t)(nxt[d] | ((uint32_t)d << 31));
                    for (int k16 = k16_0; k16 < k16_1 && ok; k16 += step) {
                        const size_t pos = nxt[d]++;
                        const size_t p0 = (size_t)pc * ppt + k16;
                        if (f >= 0) {
                            const size_t T = pos + (size_t)t0;
                            const size_t qa0 = ((T >> (f - 2)) << (f + 1)) | ((T & (((size_t)1 << (f - 2)) - 1)) << 2);
                            const uint32_t eb = (__builtin_popcount((uint32_t)qa0 & mask) & 1u) ^ page_bit(qa0) ^ (uint32_t)d;
                            const int32_t q = (int32_t)(qa0 + eb - first);
                            ok = quad_base[p0 / 4] == (q | (eb ? (1 << 30) : 0));
                        } else {
                            const size_t qa = first + 2 * pos;
                            ok = w->h_page_table[p0] == (int32_t)(2 * pos + ((__builtin_popcount((uint32_t)qa & mask) & 1u) ^ page_bit(qa) ^ (uint32_t)d));
                        }
                    }
                }
        }
        if (ok) {
            e = cudaMalloc(&w->d_unit_base, sizeof(int32_t) * unit_base.size());
            if (e == cudaSuccess) e = cudaMemcpy(w->d_unit_base, unit_base.data(), sizeof(int32_t) * unit_base.size(), cudaMemcpyHostToDevice);
            if (e == cudaSuccess) e = cudaMalloc(&w->d_page_bits, sizeof(uint32_t) * bits.size());
            if (e == cudaSuccess) e = cudaMemcpy(w->d_page_bits, bits.data(), sizeof(uint32_t) * bits.size(), cudaMemcpyHostToDevice);
            w->closed_form = 1;
            w->hash_mask = mask;
            w->hash_first = (int)first;
            w->hash_t0 = t0;
            w->closed_bytes = sizeof(int32_t) * unit_base.size() + sizeof(uint32_t) * bits.size();
        }
    }
    w->table_bytes = w->quad_free_bit >= 0 ? sizeof(int32_t) * quad_base.size() : sizeof(int32_t) * n_pages;
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
        cudaFree(w->d_unit_base);
        cudaFree(w->d_page_bits);
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

extern "C" ag_status ag_packed_closed_form(const ag_packed_weights* w, int32_t* enabled, uint32_t* mask, size_t* table_bytes,
                                           size_t* closed_bytes) {
    if (!w || !enabled) return AG_ERR_ARG;
    *enabled = w->closed_form;
    if (mask) *mask = w->hash_mask;
    if (table_bytes) *table_bytes = w->table_bytes;
    if (closed_bytes) *closed_bytes = w->closed_bytes;
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
    if ((tile_m != 16 && tile_m != 32 && tile_m != 64 && tile_m != 128 && !dense) || (N_expert % (dense ? 256 : SK_BN)) || (K % 8)) return AG_ERR_ARG;
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
    d->a_blocks = (!dense && K % SK_BK == 0) ? 1 : 0;
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
        if (!(d->a_blocks ? encode_a_slabs(&ha[g], base, view_rows, K, a_box_rows, sk_agrp((int)a_box_rows))
                          : encode_2d(&ha[g], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, view_rows, K, SK_BK, a_box_rows))) {
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
            const int wk = SK_SLABS * SK_BK;   // k rows per weight copy (both the decode-shaped and the block-pair kernel fill a stage with two k-slabs)
            const bool ok = d->w_blocks ? encode_b_blocks(&hw[g], B_list[g], K, N_expert, wk, 2)
                                        : encode_2d(&hw[g], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B_list[g], K, N_expert, 64, wk);
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
    return gemm_skinny_dispatch(d->A_all, nullptr, W, d->C_all, h[H_M], h[H_N], h[H_K], plan, plan->d_partial,
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
    cudaFree(w->d_unit_base);
    cudaFree(w->d_page_bits);
    delete w;
}

extern "C" ag_status gemm_persistent_packed(const void* A, const ag_packed_weights* W, void* Cout, int M, int N, int K,
                                            const ag_plan* plan, void* cuda_stream) {
    if (!A || !W || !Cout || !plan) return AG_ERR_ARG;
    if (plan->header[H_TILE_M] == 256)  // dense plan of block pairs over packed B panels
        return gemm_pair_dispatch(A, nullptr, W, Cout, M, N, K, plan, reinterpret_cast<cudaStream_t>(cuda_stream));
    return gemm_skinny_dispatch(A, nullptr, W, Cout, M, N, K, plan, plan->d_partial,
                                reinterpret_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the decode-shaped GEMM.
//
// Some callers must not allocate device memory at the moment they need the GEMM: an inference
// server that has handed every free byte of the GPU to its own arena (cudaMalloc simply fails
// there), a request loop with a latency budget that an allocator call would break, or code
// running between other libraries' strict "no allocation after start-up" phases.  For them the
// split-K workspace lives in the library image itself: a fixed array in device memory.  The CUDA
// runtime places the library's device code on a GPU when it is first used there (lazy module
// loading), so the array starts to exist on a GPU with the first call made on it - which is why that
// first call belongs at start-up, while memory is still to be had - and stays until the process ends.
//
// The array's name is only a host-side handle; the address the kernel needs is asked from the
// runtime once per device (cudaGetSymbolAddress, with that device current) and remembered.
constexpr size_t kNoAllocSemBytes = 16 * 1024;                   // head of the array, unused (see below)
constexpr size_t kNoAllocPartialBytes = 8u * 1024 * 1024;        // 2 Mi fp32 partial sums
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocSemBytes + kNoAllocPartialBytes];

namespace {
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[64] = {nullptr};   // device address of g_noalloc_scratch, per device ordinal
}  // namespace

extern "C" ag_status gemm_persistent_noalloc(const void* A, const void* B, void* Cout, int M, int N, int K,
                                             const ag_plan* plan, void* cuda_stream) {
    if (!A || !B || !Cout || !plan) return AG_ERR_ARG;
    {
        const ag_status cap = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
        if (cap != AG_OK) return cap;
    }
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
    // the first kNoAllocSemBytes of the array are not used (they held arrival counters when the last unit of a tile
    // added the slices); the slices start behind them as before
    float* partial = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + kNoAllocSemBytes);
    return gemm_skinny_dispatch(A, B, nullptr, Cout, M, N, K, plan, partial, stream, nullptr);
}
