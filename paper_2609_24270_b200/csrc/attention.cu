// Grouped-query attention decode (one query token per request) under the same scheduler as the GEMMs: one
// persistent block per planned SM, work unit = (request, KV head), the unit's key/value pages stored in chunks of
// the die that runs it (Section 7.1.2 of the paper: attention is one of the kernels it schedules NUMA-aware; its
// workload appendix fixes decode at S_q = 1, GQA at 8 KV heads, head dimension 128).
//
// Per unit (G = H_q / H_kv query rows, L keys, D = 128):
//     S^T[key][q] = K[key][:] . Q[q][:]          tcgen05.mma, key tile (128 keys) on the M side, Q on the N side (16)
//     P = exp((S - max) / sqrt(D))                softmax warps, one thread per key of a tile, scores in tensor memory
//     O^T[d][q]  = sum_key V[key][d] P[q][key]    tcgen05.mma, d on the M side, keys contracted; P as bf16 hi + lo parts
//     O[q][:] /= sum_key P[q][key]                epilogue
// Requests with more than 1024 keys are cut into chunks of 1024 keys, one unit per (request, KV head, chunk): such a
// unit leaves its unnormalised outputs, its score maximum and its sum of probabilities in a workspace, and a second
// kernel (k_attn_combine) puts the chunks of a (request, KV head) together.
// The KV cache is packed once (ag_kv_pack) into 4 KB pages in the MMA's no-swizzle operand order - K pages hold
// [128 keys x 16 d], V pages [128 d x 16 keys] - four pages of a 64-wide contraction slab per group of same-die
// chunks (or four consecutive chunks for the interleaved placement), so a 128-key tile of K or of V is one 32 KB
// stage filled by two strided copies.  K tiles of unit i+1 are streamed before the V tiles of unit i, so that the
// softmax of unit i runs while the scores of unit i+1 are computed.
#include <cuda_bf16.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "persist.cuh"

namespace ag {

constexpr int AT_D = 128;                 // head dimension
constexpr int AT_TILE = 128;              // keys per tile
constexpr int AT_NQ = 16;                 // query rows of the MMA's N side (G <= 8 real ones)
constexpr int AT_MAXG = 8;
constexpr int AT_MAXT = 8;                // tiles per unit: L <= 1024
constexpr int AT_STAGES = 6;
constexpr int AT_STAGE_BYTES = 32 * 1024; // one K or V tile
constexpr int AT_NPROD = 3;
constexpr int AT_THREADS = (2 + kEpiWarps + AT_NPROD) * 32;
constexpr int AT_Q_BYTES = AT_NQ * AT_D * 2;        // 4 KB
constexpr int AT_NP = 2 * AT_MAXG;         // rows of a probability tile: 8 hi parts, 8 lo parts (one MMA adds both)
constexpr int AT_P_BYTES = AT_NP * AT_TILE * 2;     // 4 KB
constexpr int AT_PSLOTS = 4;
constexpr int AT_PBATCH = 1;               // probability tiles written per fence (two per fence measured equal at 4 tiles per unit, 10 % slower at 8)
constexpr int AT_CTL_BYTES = 2048;
constexpr int AT_SMEM_BYTES = AT_STAGES * AT_STAGE_BYTES + 2 * AT_Q_BYTES + AT_PSLOTS * AT_P_BYTES + 1024 + AT_CTL_BYTES;
constexpr uint32_t AT_SCOLS = AT_MAXT * AT_NQ;      // score columns of one unit buffer (128)
constexpr uint32_t AT_BUFCOLS = AT_SCOLS + AT_NP;   // + output columns (hi-part and lo-part sums)
constexpr uint32_t AT_TMEM_COLS = 512;

struct AttnCtl {
    uint64_t kv_full[AT_STAGES], kv_empty[AT_STAGES];
    uint64_t q_full[2], q_empty[2];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[AT_PSLOTS], p_empty[AT_PSLOTS];
    uint64_t o_full[2], o_empty[2];
    uint64_t sched_full[kRing], sched_empty[kRing];
    uint64_t mma_drain;
    int ring[kRing];
    int ring_pages[kRing][4 * AT_MAXT];   // the page-list words of the unit in ring[r] (see AttnArgs::quad_of)
    uint32_t tmem_base;
    int abort_flag;
    int member;
    int4 quick;
    float red_max[kEpiWarps][AT_MAXG];
    float red_sum[2][kEpiWarps][AT_MAXG];
    float unit_max[2][AT_MAXG];           // score maximum (times log2 e / sqrt D) of the unit in buffer j, for chunked requests
};

static_assert(sizeof(AttnCtl) <= AT_CTL_BYTES, "control block does not fit its share of shared memory");

struct AttnArgs {
    const uint8_t* pages;         // packed KV buffer
    const int32_t* quad_of;       // [units][4 T]: per tile K slab 0, K slab 1, V slab 0, V slab 1: base chunk | class << 30
    const int32_t* kv_len;        // [B] or null
    float* O;                     // [B][H_q][128]
    int H_kv, G, T, L;            // T: tiles of a full unit (at most AT_MAXT)
    int n_chunks, T_total;        // units per (request, KV head); tiles of a whole request
    float* o_part;                // [units][AT_MAXG][128] unnormalised outputs (n_chunks > 1)
    float2* stats;                // [units][AT_MAXG] (maximum, sum) (n_chunks > 1)
    float scale_log2e;            // log2(e) / sqrt(D)
    int release_next;             // 1: let the next launch on the stream start while this one is still running
    int stages;                   // key/value stages in use (3 .. AT_STAGES): the bytes this block keeps in flight
};

__device__ __forceinline__ float ex2_approx(float v) {      // 2^v, relative error 2^-22; 2^-inf = 0
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// keys of unit u = (request b, KV head h, chunk c), u = (b H_kv + h) n_chunks + c: those of the request's first
// kv_len[b] keys that fall into the chunk
__device__ __forceinline__ int unit_keys(const AttnArgs& x, int u) {
    const int bh = u / x.n_chunks, c = u - bh * x.n_chunks;
    const int len = x.kv_len ? min(x.L, max(0, x.kv_len[bh / x.H_kv])) : x.L;
    return min(AT_MAXT * AT_TILE, max(0, len - c * AT_MAXT * AT_TILE));
}
__device__ __forceinline__ int unit_tiles(const AttnArgs& x, int u) { return (unit_keys(x, u) + AT_TILE - 1) / AT_TILE; }

__global__ void __launch_bounds__(AT_THREADS, 1)
k_attn_decode(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_g0,
              const __grid_constant__ CUtensorMap tm_g1, const PersistParams p, const AttnArgs x) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t q_base = base + AT_STAGES * AT_STAGE_BYTES;
    const uint32_t p_base = q_base + 2 * AT_Q_BYTES;
    AttnCtl* ctl = reinterpret_cast<AttnCtl*>(smem + AT_STAGES * AT_STAGE_BYTES + 2 * AT_Q_BYTES + AT_PSLOTS * AT_P_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int my_sm = (int)smid();
    // overlap_launches: the launch that follows on the stream may be scheduled as soon as every block of this one has
    // got this far; its blocks move in as SMs become free
    if (x.release_next && tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        ctl->abort_flag = 0;
        const int4 qk = p.quick[my_sm];
        ctl->quick = qk;
        ctl->member = qk.x >= 0 && atomicMax(&p.claimed[qk.x], p.epoch) < p.epoch;
    } else if (tid == 64) {
        for (int i = 0; i < AT_STAGES; ++i) {
            mbar_init(smem_u32(&ctl->kv_full[i]), 1);
            mbar_init(smem_u32(&ctl->kv_empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->q_full[i]), 1);
            mbar_init(smem_u32(&ctl->q_empty[i]), 1);
            mbar_init(smem_u32(&ctl->s_full[i]), 1);
            mbar_init(smem_u32(&ctl->s_empty[i]), kEpiWarps);
            mbar_init(smem_u32(&ctl->o_full[i]), 1);
            mbar_init(smem_u32(&ctl->o_empty[i]), kEpiWarps);
        }
        for (int i = 0; i < AT_PSLOTS; ++i) {
            mbar_init(smem_u32(&ctl->p_full[i]), kEpiWarps);
            mbar_init(smem_u32(&ctl->p_empty[i]), 1);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&ctl->sched_full[i]), 1);
            mbar_init(smem_u32(&ctl->sched_empty[i]), 1 + kEpiWarps + AT_NPROD);
        }
        mbar_init(smem_u32(&ctl->mma_drain), 1);
        mbar_fence_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_g0);
    }
    // the probability tiles: rows of query rows that do not exist stay zero for the whole launch
    for (int i = tid; i < AT_PSLOTS * AT_P_BYTES / 4; i += AT_THREADS)
        reinterpret_cast<uint32_t*>(smem + AT_STAGES * AT_STAGE_BYTES + 2 * AT_Q_BYTES)[i] = 0u;
    fence_proxy_async_smem();
    __syncthreads();
    const int4 quick = ctl->quick;
    const int slot = quick.x;
    if (!ctl->member) {
        if (slot < 0) wait_until_manned(p);
        return;
    }
    const uint64_t limit = p.wait_limit_ns;
    uint32_t tmem_base = 0;
    if (warp >= 1 && warp < 2 + kEpiWarps) {
        if (warp == 1) {
            tmem_alloc(smem_u32(&ctl->tmem_base), AT_TMEM_COLS);
            tmem_relinquish();
        }
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"((1 + kEpiWarps) * 32) : "memory");
        tc_fence_after();
        tmem_base = ctl->tmem_base;
    }

    if (warp == 0) {
        // ------------------------------------------------ scheduler + query copies (lane 0)
        UnitSource src(p, slot, lane, quick.y, quick.z, quick.w);
        uint32_t it = 0, nq = 0;     // ring entries pushed; units with keys so far (they alternate the two buffers)
        int ok = 1;
        while (ok) {
            int u;
            if (p.static_assign) {
                u = src.next_listed(lane);
                while (u < 0 && ok) {
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
            // the unit's page-list words travel with it through the ring (one coalesced load here, several units ahead of
            // the copies, instead of a dependent load in front of every copy)
            int page_word = 0;
            if (u >= 0) {
                const int bh = u / x.n_chunks, c = u - bh * x.n_chunks;
                if (lane < 4 * min(AT_MAXT, x.T_total - c * AT_MAXT)) page_word = x.quad_of[((size_t)bh * x.T_total + c * AT_MAXT) * 4 + lane];
            }
            {
                const int r = it % kRing;
                int w_ok = 1;
                if (lane == 0 && !mbar_wait_idle(smem_u32(&ctl->sched_empty[r]), ((it / kRing) & 1) ^ 1, abort_flag, limit)) {
                    report_timeout(p, 1);
                    w_ok = 0;
                }
                ok = __shfl_sync(0xffffffffu, w_ok, 0);
                if (ok) ctl->ring_pages[r][lane] = page_word;
                __syncwarp();
            }
            if (ok && lane == 0) {
                const int r = it % kRing;
                {
                    ctl->ring[r] = u;
                    if (p.unit_times && u >= 0) p.unit_times[2 * u] = globaltimer_ns();
                    mbar_arrive(smem_u32(&ctl->sched_full[r]));
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ++it;
            if (!ok || u < 0) break;
            if (unit_tiles(x, u) == 0) continue;
            if (lane == 0) {
                const int j = nq & 1;
                if (!mbar_wait_idle(smem_u32(&ctl->q_empty[j]), ((nq >> 1) & 1) ^ 1, abort_flag, limit)) {
                    report_timeout(p, 2);
                    ok = 0;
                } else {
                    // the G query rows of the unit's KV head (G consecutive rows of the [B H_q][128] matrix) and whatever
                    // follows them up to 16 rows: the extra rows only produce columns nobody reads
                    const uint32_t bar = smem_u32(&ctl->q_full[j]);
                    // the queries are the product of the launch before this one: with overlapping launches they are
                    // read only after it has completed (the key/value pages are the caller's promise)
                    if (nq == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
                    mbar_expect_tx(bar, AT_Q_BYTES);
                    tma_load_3d(q_base + j * AT_Q_BYTES, &tm_q, bar, 0, (u / x.n_chunks) * x.G, 0);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ++nq;
        }
    } else if (warp >= 2 + kEpiWarps) {
        // ------------------------------------------------ key/value copies.  Order of the stream: K tiles of the first
        // unit; then, unit by unit, the K tiles of the next unit followed by the V tiles of the one before.
        const int pw = warp - (2 + kEpiWarps);
        const uint64_t stream_policy = l2_policy_evict_first();
        uint32_t q_run = 0;          // stages issued by all copy warps together so far
        const uint32_t n_st = (uint32_t)x.stages;
        int prev_u = -1, prev_t = 0;
        int ok = 1;
        int words_cur = 0, words_prev = 0;   // lane l: word l of the page lists of the unit just taken off the ring / the one before
        auto copy_tiles = [&](int words, int n_t, int v_part) {
            // this warp's stages among the next n_t: ordinals q_run .. q_run + n_t - 1, those = pw mod AT_NPROD
            for (int t = 0; t < n_t && ok; ++t) {
                const uint32_t q = q_run + (uint32_t)t;
                if ((int)(q % AT_NPROD) != pw) continue;
                const uint32_t st = q % n_st, ph = ((q / n_st) & 1) ^ 1;
                const int entry = __shfl_sync(0xffffffffu, words, t * 4 + v_part * 2 + (lane & 1));
                if (lane == 0) {
                    if (!mbar_wait(smem_u32(&ctl->kv_empty[st]), ph, abort_flag, limit)) {
                        report_timeout(p, 2);
                        ok = 0;
                    } else {
                        mbar_expect_tx(smem_u32(&ctl->kv_full[st]), AT_STAGE_BYTES);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (lane < 2) {
                    const uint32_t dst = base + st * AT_STAGE_BYTES + lane * (AT_STAGE_BYTES / 2);
                    const uint32_t bar = smem_u32(&ctl->kv_full[st]);
                    const int cls = (entry >> 30) & 3, q0 = entry & 0x3fffffff;
                    if (cls == 2) bulk_load_hint(dst, x.pages + (size_t)q0 * AG_CHUNK_BYTES, AT_STAGE_BYTES / 2, bar, stream_policy);
                    else tma_load_5d_hint(dst, cls ? &tm_g1 : &tm_g0, bar, 0, 0, 0, 0, q0, stream_policy);
                }
            }
            q_run += (uint32_t)n_t;
        };
        for (uint32_t it = 0; ok; ++it) {
            const int r = it % kRing;
            int u = -1;
            if (lane == 0) {
                if (!mbar_wait_idle(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                    report_timeout(p, 8);
                    ok = 0;
                } else {
                    u = ctl->ring[r];
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            u = __shfl_sync(0xffffffffu, u, 0);
            if (!ok) break;
            __syncwarp();
            const int words_new = ctl->ring_pages[r][lane];   // read before the slot is handed back
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
            // A unit without keys has nothing to stream, but like every entry it brings the value tiles of the unit before
            // (whose outputs must not wait for a later entry: the softmax warps may be waiting for them before they take
            // the next unit off the ring).
            const int n_t = u >= 0 ? unit_tiles(x, u) : 0;
            words_cur = words_new;
            if (n_t > 0) copy_tiles(words_cur, n_t, 0);
            if (prev_u >= 0 && ok) copy_tiles(words_prev, prev_t, 1);
            words_prev = words_cur;
            prev_u = n_t > 0 ? u : -1;
            prev_t = n_t;
            if (u < 0) break;
        }
        if (!ok && lane == 0) {
            const uint64_t t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        }
    } else if (warp == 1) {
        {
            // ------------------------------------------------ MMA issuer: scores of unit i, then the outputs of unit i - 1
            // (the warp runs the loop converged and one elected lane issues the MMAs and commits: see elect_one)
            constexpr uint32_t idesc = make_idesc_bf16(128, AT_NQ, 0, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, AT_NP, 0, 0);
            static_assert(AT_NP == 16 && AT_MAXG == 8, "rows q and 8 + q of a probability tile are the two parts of query row q");
            const uint64_t dpage_t = make_smem_desc(0, 128, 256, 0);     // K and V pages: no swizzle, K-major (see ag_kv_pack)
            const uint64_t dsw_t = make_smem_desc(0, 16, 1024, 2);       // Q and P tiles: K-major, 128-byte swizzle
            const uint32_t full0 = smem_u32(&ctl->kv_full[0]), empty0 = smem_u32(&ctl->kv_empty[0]);
            uint32_t st = 0, ph = 0;
            uint32_t nq = 0;             // units with keys whose scores have been issued
            uint32_t pt = 0;             // probability tiles consumed (ring of AT_PSLOTS)
            int prev_t = 0;              // tiles of the unit whose outputs are still to be computed
            bool have_prev = false, ok = true;
            auto next_stage = [&]() -> uint32_t {
                const uint32_t s = st;
                if (++st == (uint32_t)x.stages) { st = 0; ph ^= 1; }
                return s;
            };
            for (uint32_t it = 0; ok; ++it) {
                const int r = it % kRing;
                if (!mbar_wait_all(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                    if (lane == 0) report_timeout(p, 3);
                    break;
                }
                const int u = ctl->ring[r];
                __syncwarp();       // every lane has read the entry before it is handed back
                if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                const int n_t = u >= 0 ? unit_tiles(x, u) : 0;     // 0: the end of the list, or a unit without keys
                if (n_t > 0) {
                    // ---- S^T = K Q^T for every key tile of the unit
                    const uint32_t j = nq & 1;
                    if (!mbar_wait_all(smem_u32(&ctl->s_empty[j]), ((nq >> 1) & 1) ^ 1, abort_flag, limit) ||
                        !mbar_wait_all(smem_u32(&ctl->q_full[j]), (nq >> 1) & 1, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 4);
                        break;
                    }
                    tc_fence_after();
                    const uint64_t dq = dsw_t | (uint64_t)((q_base + j * AT_Q_BYTES) >> 4);
                    for (int t = 0; t < n_t; ++t) {
                        const uint32_t phw = ph, s = next_stage();
                        if (!mbar_wait_all(full0 + s * 8, phw, abort_flag, limit)) {
                            if (lane == 0) report_timeout(p, 5);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t dk = dpage_t | (uint64_t)((base + s * AT_STAGE_BYTES) >> 4);
                        const uint32_t d_s = tmem_base + j * AT_BUFCOLS + t * AT_NQ;
                        if (elect_one()) {
#pragma unroll
                            for (int g = 0; g < AT_D / 16; ++g)   // 16 d per step: page g of the tile; Q: atom g / 4, 32 B per step
                                tc_mma_f16(d_s, dk + g * (4096u >> 4), dq + (g >> 2) * (2048u >> 4) + (g & 3) * 2, idesc, g ? 1u : 0u);
                            tc_commit(empty0 + s * 8);
                        }
                        __syncwarp();
                    }
                    if (!ok) break;
                    if (elect_one()) {
                        tc_commit(smem_u32(&ctl->s_full[j]));
                        tc_commit(smem_u32(&ctl->q_empty[j]));
                    }
                    __syncwarp();
                    ++nq;
                }
                if (have_prev) {
                    // ---- O^T += V^T P^T for every key tile of the previous unit (probabilities as hi + lo bf16 parts)
                    const uint32_t np = nq - (n_t > 0 ? 2 : 1);         // ordinal of the previous unit
                    const uint32_t j = np & 1;
                    if (!mbar_wait_all(smem_u32(&ctl->o_empty[j]), ((np >> 1) & 1) ^ 1, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 4);
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_o = tmem_base + j * AT_BUFCOLS + AT_SCOLS;
                    for (int t = 0; t < prev_t; ++t, ++pt) {
                        const uint32_t phw = ph, s = next_stage();
                        const uint32_t ps = pt % AT_PSLOTS;
                        if (!mbar_wait_all(smem_u32(&ctl->p_full[ps]), (pt / AT_PSLOTS) & 1, abort_flag, limit) ||
                            !mbar_wait_all(full0 + s * 8, phw, abort_flag, limit)) {
                            if (lane == 0) report_timeout(p, 5);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t dv = dpage_t | (uint64_t)((base + s * AT_STAGE_BYTES) >> 4);
                        const uint64_t dp = dsw_t | (uint64_t)((p_base + ps * AT_P_BYTES) >> 4);
                        if (elect_one()) {
#pragma unroll
                            for (int k8 = 0; k8 < AT_TILE / 16; ++k8)     // 16 keys per step: page k8 of the tile; P: atom k8 / 4
                                tc_mma_f16(d_o, dv + k8 * (4096u >> 4), dp + (k8 >> 2) * (2048u >> 4) + (k8 & 3) * 2, idesc_pv,
                                           (t | k8) ? 1u : 0u);
                            tc_commit(empty0 + s * 8);
                            tc_commit(smem_u32(&ctl->p_empty[ps]));
                        }
                        __syncwarp();
                    }
                    if (!ok) break;
                    if (elect_one()) tc_commit(smem_u32(&ctl->o_full[j]));
                    __syncwarp();
                }
                have_prev = n_t > 0;
                prev_t = n_t;
                if (u < 0) break;
            }
            __syncwarp();
            if (*abort_flag) {
                if (elect_one()) {
                    tc_commit(smem_u32(&ctl->mma_drain));
                    int dummy = 0;
                    mbar_wait(smem_u32(&ctl->mma_drain), 0, &dummy, 2000000ull);
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------ softmax and epilogue: thread i of the four warps = key i of a tile
        // (scores) and = output column d = i (outputs); tensor-memory lane i.  The outputs of a unit are written after the
        // probabilities of the next one, so that the wait for its last value tile is off the path to the next products.
        const int wq = warp & 3;                      // lane quarter this warp may read
        const int i_lane = wq * 32 + lane;
        const int widx = warp - 2;
        uint32_t nq = 0, pt = 0;
        bool prior_done = false, ok = true;
        const int G = x.G;
        int pend_u = -1;                              // unit whose outputs are still to be written
        auto write_outputs = [&](uint32_t np) -> bool {     // np: the unit's ordinal among the units with keys
            const uint32_t j = np & 1;
            if (!mbar_wait_warp(smem_u32(&ctl->o_full[j]), (np >> 1) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 7);
                return false;
            }
            tc_fence_after();
            uint32_t vh[8], vl[8];
            const uint32_t t_o = tmem_base + ((uint32_t)(wq * 32) << 16) + j * AT_BUFCOLS + AT_SCOLS;
            tmem_ld_32x8(t_o, vh);
            tmem_ld_32x8(t_o + AT_MAXG, vl);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->o_empty[j]));
            if (x.n_chunks == 1) {
                float* out = x.O + (size_t)pend_u * G * AT_D + i_lane;
#pragma unroll
                for (int q = 0; q < AT_MAXG; ++q) {
                    if (q < G) {
                        const float l = (ctl->red_sum[j][0][q] + ctl->red_sum[j][1][q]) + (ctl->red_sum[j][2][q] + ctl->red_sum[j][3][q]);
                        out[(size_t)q * AT_D] = __fdividef(__uint_as_float(vh[q]) + __uint_as_float(vl[q]), l);
                    }
                }
            } else {
                // a chunk of a longer request: unnormalised outputs, maximum and sum for k_attn_combine
                float* part = x.o_part + (size_t)pend_u * AT_MAXG * AT_D + i_lane;
#pragma unroll
                for (int q = 0; q < AT_MAXG; ++q) {
                    if (q < G) {
                        part[(size_t)q * AT_D] = __uint_as_float(vh[q]) + __uint_as_float(vl[q]);
                        if (i_lane == q) {
                            const float l = (ctl->red_sum[j][0][q] + ctl->red_sum[j][1][q]) + (ctl->red_sum[j][2][q] + ctl->red_sum[j][3][q]);
                            x.stats[(size_t)pend_u * AT_MAXG + q] = make_float2(ctl->unit_max[j][q], l);
                        }
                    }
                }
            }
            if (lane == 0 && wq == 0) {
                p.tile_owner[pend_u] = my_sm;
                if (p.unit_times) p.unit_times[2 * pend_u + 1] = globaltimer_ns();
                atomicAdd(&p.tile_count[pend_u], 1);
            }
            pend_u = -1;
            return true;
        };
        for (uint32_t it = 0; ok; ++it) {
            const int r = it % kRing;
            if (!mbar_wait_warp(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 6);
                break;
            }
            const int u = ctl->ring[r];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->sched_empty[r]));
            if (u < 0) break;
            const int len = unit_keys(x, u);              // keys of this unit that count
            const int n_t = (len + AT_TILE - 1) / AT_TILE;
            if (!prior_done) {      // nothing is written before everything launched earlier on the stream has completed
                asm volatile("griddepcontrol.wait;" ::: "memory");
                prior_done = true;
            }
            if (n_t == 0) {
                if (pend_u >= 0 && !(ok = write_outputs(nq - 1))) break;   // their products were issued on this entry
                if (x.n_chunks == 1) {
                    float* out = x.O + (size_t)u * G * AT_D + i_lane;
                    for (int q = 0; q < G; ++q) out[(size_t)q * AT_D] = 0.f;
                } else if (i_lane < G) {
                    x.stats[(size_t)u * AT_MAXG + i_lane] = make_float2(-INFINITY, 0.f);   // a chunk without keys: nothing to add
                }
                if (lane == 0 && wq == 0) {
                    p.tile_owner[u] = my_sm;
                    if (p.unit_times) p.unit_times[2 * u + 1] = globaltimer_ns();
                    atomicAdd(&p.tile_count[u], 1);
                }
                continue;
            }
            const uint32_t j = nq & 1;
            if (!mbar_wait_warp(smem_u32(&ctl->s_full[j]), (nq >> 1) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 7);
                break;
            }
            tc_fence_after();
            // ---- scores of this thread's key in every tile; running maximum per query row
            uint32_t sv[AT_MAXT][AT_MAXG];
            const uint32_t t_s = tmem_base + ((uint32_t)(wq * 32) << 16) + j * AT_BUFCOLS;
#pragma unroll
            for (int t = 0; t < AT_MAXT; ++t)
                if (t < n_t) tmem_ld_32x8(t_s + t * AT_NQ, sv[t]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->s_empty[j]));      // the score columns may be overwritten
            float mx[AT_MAXG];
#pragma unroll
            for (int q = 0; q < AT_MAXG; ++q) mx[q] = -INFINITY;
#pragma unroll
            for (int t = 0; t < AT_MAXT; ++t) {
                if (t < n_t) {
                    const bool valid = t * AT_TILE + i_lane < len;
#pragma unroll
                    for (int q = 0; q < AT_MAXG; ++q) {
                        if (!valid) sv[t][q] = 0xff800000u;               // -inf: a key past the request's length
                        mx[q] = fmaxf(mx[q], __uint_as_float(sv[t][q]));
                    }
                }
            }
            // warp maximum with one integer reduction per query row: floats compare like the signed integers
            // b ^ ((b >> 31) & 0x7fffffff) of their bit patterns b
#pragma unroll
            for (int q = 0; q < AT_MAXG; ++q) {
                if (q < G) {
                    const int b = __float_as_int(mx[q]);
                    const int m = __reduce_max_sync(0xffffffffu, b ^ ((b >> 31) & 0x7fffffff));
                    mx[q] = __int_as_float(m ^ ((m >> 31) & 0x7fffffff));
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < AT_MAXG; ++q)
                    if (q < G) ctl->red_max[widx][q] = mx[q];
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * 32) : "memory");
#pragma unroll
            for (int q = 0; q < AT_MAXG; ++q)
                if (q < G)
                    mx[q] = fmaxf(fmaxf(ctl->red_max[0][q], ctl->red_max[1][q]), fmaxf(ctl->red_max[2][q], ctl->red_max[3][q])) * x.scale_log2e;
            if (x.n_chunks > 1 && i_lane < G) {
#pragma unroll
                for (int q = 0; q < AT_MAXG; ++q)
                    if (q == i_lane) ctl->unit_max[j][q] = mx[q];
            }
            // ---- probabilities, tile by tile, into the ring of probability tiles: rows 0-7 the bf16 hi parts, rows
            // 8-15 the lo parts (row = query row; the rows of query rows that do not exist stay zero)
            float sum[AT_MAXG];
#pragma unroll
            for (int q = 0; q < AT_MAXG; ++q) sum[q] = 0.f;
            const uint32_t atom = (uint32_t)(i_lane >> 6) * 2048u;                 // keys 0-63 / 64-127 of the tile
            const uint32_t chunk = (uint32_t)((i_lane & 63) >> 3), within = (uint32_t)(i_lane & 7) * 2u;
            // AT_PBATCH tiles at a time: one fence and one round of barrier traffic per batch
#pragma unroll
            for (int b0 = 0; b0 < AT_MAXT; b0 += AT_PBATCH) {
                if (b0 < n_t && ok) {
                    const int nb = min(AT_PBATCH, n_t - b0);
                    int w_ok = 1;
                    if (lane == 0) {
                        for (int tt = 0; tt < nb && w_ok; ++tt)
                            w_ok = mbar_wait(smem_u32(&ctl->p_empty[(pt + tt) % AT_PSLOTS]), (((pt + tt) / AT_PSLOTS) & 1) ^ 1, abort_flag, limit);
                        if (!w_ok) report_timeout(p, 7);
                    }
                    ok = __shfl_sync(0xffffffffu, w_ok, 0) != 0;
                    if (ok) {
#pragma unroll
                        for (int tt = 0; tt < AT_PBATCH; ++tt) {
                            if (tt < nb) {
                                uint8_t* ptile = smem + AT_STAGES * AT_STAGE_BYTES + 2 * AT_Q_BYTES + ((pt + tt) % AT_PSLOTS) * AT_P_BYTES;
#pragma unroll
                                for (int q = 0; q < AT_MAXG; ++q) {
                                    if (q < G) {
                                        // masked keys: exp2(-inf) = 0
                                        const float pv = ex2_approx(fmaf(__uint_as_float(sv[b0 + tt][q]), x.scale_log2e, -mx[q]));
                                        sum[q] += pv;
                                        const __nv_bfloat16 hi = __float2bfloat16_rn(pv);
                                        const __nv_bfloat16 lo = __float2bfloat16_rn(pv - __bfloat162float(hi));
                                        const uint32_t off = atom + (uint32_t)q * 128u + ((chunk ^ (uint32_t)(q & 7)) << 4) + within;
                                        *reinterpret_cast<__nv_bfloat16*>(ptile + off) = hi;
                                        *reinterpret_cast<__nv_bfloat16*>(ptile + 1024 + off) = lo;
                                    }
                                }
                            }
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0)
                            for (int tt = 0; tt < nb; ++tt) mbar_arrive(smem_u32(&ctl->p_full[(pt + tt) % AT_PSLOTS]));
                        pt += (uint32_t)nb;
                    }
                }
            }
            if (!ok) break;
#pragma unroll
            for (int q = 0; q < AT_MAXG; ++q) {
                if (q < G) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) sum[q] += __shfl_xor_sync(0xffffffffu, sum[q], o);
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < AT_MAXG; ++q) ctl->red_sum[j][widx][q] = sum[q];
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * 32) : "memory");
            // ---- outputs of the unit before this one, while this one's value tiles stream in
            if (pend_u >= 0) ok = write_outputs(nq - 1);
            pend_u = u;
            ++nq;
        }
        if (ok && pend_u >= 0 && !*abort_flag) write_outputs(nq - 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, AT_TMEM_COLS);
    }
}

// Chunked requests: one block per (request, KV head), thread = output column d.  With m_c, l_c, O_c the maximum (in
// units of log2 e / sqrt D), the sum of probabilities and the unnormalised outputs of chunk c:
// O = sum_c 2^(m_c - m) O_c / sum_c 2^(m_c - m) l_c, m = max_c m_c; chunks without keys (l_c = 0) are left out.
__global__ void __launch_bounds__(AT_D) k_attn_combine(const float* __restrict__ o_part, const float2* __restrict__ stats,
                                                        float* __restrict__ O, int n_chunks, int G) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int bh = blockIdx.x / G, q = blockIdx.x - bh * G, d = threadIdx.x;     // one block per (request, KV head, query row)
    const float2* st = stats + (size_t)bh * n_chunks * AT_MAXG + q;
    const float* part = o_part + ((size_t)bh * n_chunks * AT_MAXG + q) * AT_D + d;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) {
        const float2 s2 = __ldcg(st + (size_t)c * AT_MAXG);
        if (s2.y > 0.f) m = fmaxf(m, s2.x);
    }
    float num = 0.f, den = 0.f;
#pragma unroll 4
    for (int c = 0; c < n_chunks; ++c) {
        const float2 s2 = __ldcg(st + (size_t)c * AT_MAXG);
        const float v = __ldcg(part + (size_t)c * AT_MAXG * AT_D);   // finite or not: only used when the chunk had keys
        if (s2.y > 0.f) {
            const float w = ex2_approx(s2.x - m);
            num = fmaf(w, v, num);
            den = fmaf(w, s2.y, den);
        }
    }
    O[((size_t)bh * G + q) * AT_D + d] = den > 0.f ? num / den : 0.f;
}

// One block per 4 KB page.  which = 0: K page (unit, tile t, d group g): element (n = key, k = d) = K[u][128 t + n][16 g + k];
// which = 1: V page (unit, tile t, key group j): element (n = d, k = key) = V[u][128 t + 16 j + k][n].  Both in the MMA's
// no-swizzle K-major order: byte (n / 8) * 256 + (k / 8) * 128 + (n % 8) * 16 + (k % 8) * 2.
__global__ void k_pack_kv(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V, int L, int T,
                          const int32_t* __restrict__ page_chunk, uint8_t* __restrict__ dst) {
    const int page = blockIdx.x;                   // ((u * T + t) * 2 + which) * 8 + g
    const int g = page & 7, which = (page >> 3) & 1, ut = page >> 4;
    const int u = ut / T, t = ut - u * T;
    const int n = threadIdx.x;                     // 128 threads
    uint16_t v[16];
    if (which == 0) {
        const uint16_t* src = K + ((size_t)u * L + (size_t)t * AT_TILE + n) * AT_D + g * 16;
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = src[k];
    } else {
        const uint16_t* src = V + ((size_t)u * L + (size_t)t * AT_TILE + g * 16) * AT_D + n;
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = src[(size_t)k * AT_D];
    }
    uint8_t* out = dst + (size_t)page_chunk[page] * AG_CHUNK_BYTES + (n / 8) * 256 + (n % 8) * 16;
    uint4 lo, hi;
    lo.x = v[0] | (v[1] << 16); lo.y = v[2] | (v[3] << 16); lo.z = v[4] | (v[5] << 16); lo.w = v[6] | (v[7] << 16);
    hi.x = v[8] | (v[9] << 16); hi.y = v[10] | (v[11] << 16); hi.z = v[12] | (v[13] << 16); hi.w = v[14] | (v[15] << 16);
    *reinterpret_cast<uint4*>(out) = lo;
    *reinterpret_cast<uint4*>(out + 128) = hi;
}

// One block per (request, KV head): writes the key and value row of one new token (position pos[b] of the request)
// into the pages, in the same byte order as k_pack_kv.  Thread = dimension d.
__global__ void __launch_bounds__(AT_D) k_kv_append(const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                                                     const int32_t* __restrict__ pos, int H_kv, int L, int T,
                                                     const int32_t* __restrict__ page_chunk, uint8_t* __restrict__ dst) {
    const int bh = blockIdx.x, d = threadIdx.x;
    const int at = pos[bh / H_kv];
    if (at < 0 || at >= L) return;                       // no room (or no token) for this request
    const int t = at / AT_TILE, n = at % AT_TILE;
    const size_t page0 = ((size_t)bh * T + t) * 16;      // the tile's 8 K pages, then its 8 V pages
    // K page g = d / 16 holds [128 keys x 16 d]: element (key n, k = d % 16)
    {
        const int g = d >> 4, k = d & 15;
        uint8_t* out = dst + (size_t)page_chunk[page0 + g] * AG_CHUNK_BYTES + (n / 8) * 256 + (k / 8) * 128 + (n % 8) * 16 + (k % 8) * 2;
        *reinterpret_cast<uint16_t*>(out) = k_new[(size_t)bh * AT_D + d];
    }
    // V page j = n / 16 holds [128 d x 16 keys]: element (d, k = n % 16)
    {
        const int j = n >> 4, k = n & 15;
        uint8_t* out = dst + (size_t)page_chunk[page0 + 8 + j] * AG_CHUNK_BYTES + (d / 8) * 256 + (k / 8) * 128 + (d % 8) * 16 + (k % 8) * 2;
        *reinterpret_cast<uint16_t*>(out) = v_new[(size_t)bh * AT_D + d];
    }
}

}  // namespace ag

using namespace ag;

struct ag_kv_cache {
    int B, H_kv, L, T, placement, free_bit;
    int n_chunks;                        // units per (request, KV head): chunks of AT_MAXT tiles
    const uint8_t* dst;
    size_t dst_bytes;
    int32_t* d_quad_of;                  // device [B H_kv][4 T]
    int32_t* d_page_chunk;               // device [B H_kv][T][16]: chunk of every page (8 K pages, 8 V pages per tile)
    float* d_part;                       // device [units][AT_MAXG][128] (n_chunks > 1): unnormalised outputs of the chunks
    float2* d_stats;                     // device [units][AT_MAXG] (n_chunks > 1)
    std::vector<int32_t> h_quad_of;
    CUtensorMap tm_quad[2];
    double local_fraction;               // share of the pages that sit on the die that runs their unit
};

extern "C" void ag_kv_destroy(ag_kv_cache* kv) {
    if (!kv) return;
    cudaFree(kv->d_quad_of);
    cudaFree(kv->d_page_chunk);
    cudaFree(kv->d_part);
    cudaFree(kv->d_stats);
    delete kv;
}

extern "C" ag_status ag_kv_pack(const void* K, const void* V, int B, int H_kv, int L, int D, const ag_plan* plan,
                                const ag_affinity_map* amap, void* dst, size_t dst_bytes, int placement, ag_kv_cache** out) {
    if (!K || !V || !plan || !amap || !dst || !out || B < 1 || H_kv < 1 || D != AT_D || L < AT_TILE || (L % AT_TILE) ||
        L > (1 << 20) || placement < 0 || placement > 2)
        return AG_ERR_ARG;
    *out = nullptr;
    const int T = L / AT_TILE;                                  // tiles of a request
    const int n_chunks = (T + AT_MAXT - 1) / AT_MAXT;           // units per (request, KV head)
    const long long n_bh = (long long)B * H_kv, n_units = n_bh * n_chunks;
    if (n_units != plan->lay.n_units || plan->header[H_KSPLITS] != 1) return AG_ERR_ARG;
    if (amap->base != dst || amap->bytes != dst_bytes) return AG_ERR_STALE_AMAP;
    // slabs (groups of four pages) per (request, KV head); slab i belongs to tile (i % quads_per_bh) / 4 of (request, KV
    // head) i / quads_per_bh, i.e. to unit (i / quads_per_bh) n_chunks + tile / AT_MAXT
    const size_t quads_per_bh = 4 * (size_t)T, n_quads = quads_per_bh * (size_t)n_bh;
    auto unit_of_quad = [&](size_t i) -> size_t { return (i / quads_per_bh) * n_chunks + ((i % quads_per_bh) / 4) / AT_MAXT; };
    // die of every unit from the plan's die queues
    const PlanLayout& lay = plan->lay;
    const int32_t* img = plan->h_image.data();
    std::vector<uint8_t> unit_die(lay.n_units, 0);
    for (int e = img[lay.die_q_off() + 1]; e < lay.n_units; ++e) unit_die[img[lay.die_q() + e]] = 1;
    ag_kv_cache* kv = new (std::nothrow) ag_kv_cache();
    if (!kv) return AG_ERR_NOMEM;
    kv->B = B; kv->H_kv = H_kv; kv->L = L; kv->T = T; kv->placement = placement; kv->free_bit = -1; kv->n_chunks = n_chunks;
    kv->dst = (const uint8_t*)dst; kv->dst_bytes = dst_bytes; kv->d_quad_of = nullptr; kv->d_page_chunk = nullptr; kv->d_part = nullptr; kv->d_stats = nullptr;
    kv->h_quad_of.resize(n_quads);
    size_t on_die = 0;
    if (placement == 2) {
        // interleaved: the hardware's default - four consecutive chunks per slab
        if (n_quads * 4 > amap->n_chunks) { delete kv; return AG_ERR_ARG; }
        for (size_t i = 0; i < n_quads; ++i) {
            kv->h_quad_of[i] = (int32_t)(4 * i) | (2 << 30);
            for (int c = 0; c < 4; ++c) on_die += amap->h_die_of_chunk[4 * i + c] == unit_die[unit_of_quad(i)];
        }
    } else {
        // groups of four same-die chunks, as for packed weights (see ag_pack_weights_ex)
        uint32_t mask = 0;
        size_t violations = 0;
        int f = -1;
        if (ag_affinity_fit_hash(amap, &mask, &violations) == AG_OK && (mask & 3u) == 3u && violations * 50 <= amap->n_chunks)
            for (int b = 2; b < 9 && f < 0; ++b)
                if (!((mask >> b) & 1u)) f = b;
        if (f < 0) { delete kv; return AG_ERR_NOISY_PROBE; }   // the map shows no hash with a free bit: no such groups
        const size_t F = (size_t)1 << f;
        const size_t first = ((uintptr_t)dst / AG_CHUNK_BYTES) % 512;
        std::vector<int32_t> groups[2];
        for (size_t q = 0; q + F + 3 < amap->n_chunks; ++q) {
            const size_t qa = first + q;
            if ((qa & F) || (qa & 3) > 1) continue;
            const size_t a = (qa & 3) == 0 ? 3 : 1;
            const uint8_t d0 = amap->h_die_of_chunk[q];
            if (amap->h_die_of_chunk[q + a] == d0 && amap->h_die_of_chunk[q + F] == d0 && amap->h_die_of_chunk[q + F + a] == d0)
                groups[d0].push_back((int32_t)q | (a == 1 ? (1 << 30) : 0));
        }
        size_t nxt[2] = {0, 0};
        for (size_t i = 0; i < n_quads; ++i) {
            const int d = unit_die[unit_of_quad(i)] ^ (placement == 1 ? 1 : 0);
            if (nxt[d] >= groups[d].size()) { delete kv; return AG_ERR_ARG; }   // destination too small for this die's share
            kv->h_quad_of[i] = groups[d][nxt[d]++];
        }
        on_die = placement == 0 ? n_quads * 4 : 0;
        kv->free_bit = f;
        EncodeTiledFn enc = get_encode_tiled();
        for (int cls = 0; cls < 2; ++cls) {
            const cuuint64_t a = cls == 0 ? 3 : 1;
            cuuint64_t dims[5] = {128, 16, 2, 2, (cuuint64_t)amap->n_chunks};
            cuuint64_t strides[4] = {256, a * AG_CHUNK_BYTES, (cuuint64_t)F * AG_CHUNK_BYTES, AG_CHUNK_BYTES};
            cuuint32_t box[5] = {128, 16, 2, 2, 1};
            cuuint32_t estr[5] = {1, 1, 1, 1, 1};
            if (!enc || enc(&kv->tm_quad[cls], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, dst, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
                delete kv;
                return AG_ERR_CUDA;
            }
        }
    }
    kv->local_fraction = (double)on_die / (double)(n_quads * 4);
    // chunk of every page: the four pages of a slab go to the group's chunks q, q + a, q + F, q + F + a (a group of the
    // interleaved placement: q .. q + 3)
    std::vector<int32_t> page_chunk(n_quads * 4);
    for (size_t i = 0; i < n_quads; ++i) {
        const int32_t e = kv->h_quad_of[i];
        const int cls = (e >> 30) & 3;
        const int32_t q = e & 0x3fffffff;
        const int32_t a = cls == 2 ? 1 : (cls == 1 ? 1 : 3), Fq = cls == 2 ? 2 : (1 << kv->free_bit);
        // quad i = (unit, tile t, part (K slab 0, K slab 1, V slab 0, V slab 1)); its pages g = 4 (part & 1) .. + 3 of the
        // tile's K or V pages
        const size_t ut = i / 4, part = i % 4;
        const size_t page0 = (ut * 2 + (part >> 1)) * 8 + (part & 1) * 4;
        page_chunk[page0 + 0] = q;
        page_chunk[page0 + 1] = q + a;
        page_chunk[page0 + 2] = q + Fq;
        page_chunk[page0 + 3] = q + Fq + a;
    }
    int32_t*& d_chunk = kv->d_page_chunk;
    cudaError_t e = cudaMalloc(&kv->d_quad_of, sizeof(int32_t) * n_quads);
    if (e == cudaSuccess) e = cudaMemcpy(kv->d_quad_of, kv->h_quad_of.data(), sizeof(int32_t) * n_quads, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && n_chunks > 1) e = cudaMalloc(&kv->d_part, sizeof(float) * (size_t)n_units * AT_MAXG * AT_D);
    if (e == cudaSuccess && n_chunks > 1) e = cudaMalloc(&kv->d_stats, sizeof(float2) * (size_t)n_units * AT_MAXG);
    if (e == cudaSuccess) e = cudaMalloc(&d_chunk, sizeof(int32_t) * page_chunk.size());
    if (e == cudaSuccess) e = cudaMemcpy(d_chunk, page_chunk.data(), sizeof(int32_t) * page_chunk.size(), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        k_pack_kv<<<(unsigned)page_chunk.size(), 128>>>((const uint16_t*)K, (const uint16_t*)V, L, T, d_chunk, (uint8_t*)dst);
        count_launch();
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        ag_kv_destroy(kv);
        return cuda_fail(e);
    }
    *out = kv;
    return AG_OK;
}

extern "C" ag_status ag_kv_append(ag_kv_cache* kv, const void* k_new, const void* v_new, const int32_t* pos, void* cuda_stream) {
    if (!kv || !k_new || !v_new || !pos) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    k_kv_append<<<(unsigned)(kv->B * kv->H_kv), AT_D, 0, stream>>>((const uint16_t*)k_new, (const uint16_t*)v_new, pos, kv->H_kv, kv->L,
                                                                    kv->T, kv->d_page_chunk, const_cast<uint8_t*>(kv->dst));
    count_launch();
    AG_CUDA(cudaGetLastError());
    return AG_OK;
}

extern "C" ag_status ag_kv_info(const ag_kv_cache* kv, int32_t* group_free_bit, double* local_fraction) {
    if (!kv) return AG_ERR_ARG;
    if (group_free_bit) *group_free_bit = kv->free_bit;
    if (local_fraction) *local_fraction = kv->local_fraction;
    return AG_OK;
}

extern "C" ag_status attention_decode_persistent(const void* Q, const ag_kv_cache* kv, const int32_t* kv_len, void* O, int B,
                                                 int H_q, const ag_plan* plan, void* cuda_stream) {
    if (!Q || !kv || !O || !plan || B != kv->B || H_q < kv->H_kv || (H_q % kv->H_kv)) return AG_ERR_ARG;
    const int G = H_q / kv->H_kv;
    if (G > AT_MAXG || (((uintptr_t)Q | (uintptr_t)O) & 15u)) return AG_ERR_ARG;
    const int32_t* h = plan->header;
    if ((long long)B * kv->H_kv * kv->n_chunks != plan->lay.n_units || h[H_KSPLITS] != 1) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if ((st = refuse_capture(stream)) != AG_OK) return st;
    if ((st = renew_epochs_if_needed(plan, stream)) != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (n_sm != plan->lay.n_sm) return AG_ERR_ARG;
    // Q as [2 d halves][B H_q rows][64 d]: one box of (64, 16 rows, 2) is a unit's query rows in the swizzled K-major order
    CUtensorMap tm_q;
    if (!encode_a_slabs(&tm_q, Q, (uint64_t)B * H_q, AT_D, AT_NQ, 2)) return AG_ERR_CUDA;
    CUtensorMap tm0, tm1;
    if (kv->placement == 2) { tm0 = tm_q; tm1 = tm_q; } else { tm0 = kv->tm_quad[0]; tm1 = kv->tm_quad[1]; }
    static std::atomic<unsigned long long> attr_done{0};
    const cudaError_t attr_err = once_per_device(attr_done, [] {
        return cudaFuncSetAttribute(k_attn_decode, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err);
    AttnArgs x;
    memset(&x, 0, sizeof x);
    x.pages = kv->dst;
    x.quad_of = kv->d_quad_of;
    x.kv_len = kv_len;
    x.O = (float*)O;
    x.H_kv = kv->H_kv; x.G = G; x.T = std::min(kv->T, AT_MAXT); x.L = kv->L;
    x.n_chunks = kv->n_chunks; x.T_total = kv->T;
    x.o_part = kv->d_part; x.stats = kv->d_stats;
    x.scale_log2e = 1.4426950408889634f / sqrtf((float)AT_D);
    x.stages = ring_stages_for(plan, AT_STAGES, AT_NPROD, false, true);
    PersistParams gp = make_persist_params(plan, h[H_M], h[H_N], h[H_K]);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(plan->grid_blocks > 0 ? plan->grid_blocks : plan->lay.n_sm);
    cfg.blockDim = dim3(AT_THREADS);
    cfg.dynamicSmemBytes = AT_SMEM_BYTES;
    cfg.stream = stream;
    const bool overlap = plan->policy.overlap_launches && h[H_STATIC] && plan->grid_blocks == 0;
    if (overlap && plan->lay.b < plan->lay.n_sm) gp.manned_wait_ns = gp.wait_limit_ns;   // see gemm_skinny_dispatch
    x.release_next = overlap ? 1 : 0;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, k_attn_decode, tm_q, tm0, tm1, gp, x);
    if (le != cudaSuccess) return launch_failed(plan, le);
    count_launch();
    if (kv->n_chunks > 1) {
        // requests of more than AT_MAXT tiles: the chunks' partial results are put together by a second kernel, which may
        // become resident while the first one runs and waits for its completion on the device
        cudaLaunchConfig_t cc;
        memset(&cc, 0, sizeof cc);
        cc.gridDim = dim3((unsigned)(B * kv->H_kv * G));
        cc.blockDim = dim3(AT_D);
        cc.stream = stream;
        cudaLaunchAttribute ca[1];
        ca[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        ca[0].val.programmaticStreamSerializationAllowed = 1;
        cc.attrs = ca;
        cc.numAttrs = 1;
        AG_CUDA(cudaLaunchKernelEx(&cc, k_attn_combine, (const float*)kv->d_part, (const float2*)kv->d_stats, (float*)O, kv->n_chunks, G));
        count_launch();
    }
    return AG_OK;
}
