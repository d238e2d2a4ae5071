// sched_build: the asymmetry-aware plan builder (Section 7.1.2 / 7.4.1 of the paper) as CUDA
// kernels.  All arithmetic is integer.  The plan image is produced on the device in the
// export layout and stays there for gemm_persistent; the host only marshals arguments.
//
// Steps (same order as the paper's principles are applied):
//   1. raster order of the work units (closed form, raster_unit()).
//   2. SM set: oblivious (lowest ids or seeded Fisher-Yates subset) or die-compact
//      (primary die first, whole TPCs dealt round-robin over that die's GPCs).
//   3. per-die SM counts and ranks.       4. quotas proportional to the SM count per die.
//   5. unit -> die (modulo / contiguous bands / byte-affinity margins, greedy under quotas).
//   6. static per-SM lists.               7. image = header + arrays.
#include <string.h>

#include <new>

#include "internal.h"

namespace ag {

struct OperandDev {
    int present, layout, elem_bytes, pad;
    long long offset, row_stride;
    const int32_t* page_table;  // device
};
struct PolicyDev {
    int kind, M, N, K, tile_m, tile_n, k_splits, k_unit, raster_group, preferred_die, invert, static_assign;
    int sm_select, pair_lists, cluster_size, die_quota;
    unsigned long long seed;
    long long min_margin;
    unsigned long long avoid[4];
    OperandDev a, b, c;
};

__host__ __device__ inline unsigned long long mix64(unsigned long long x) {
    x += 0x9E3779B97F4A7C15ull;
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

__device__ inline int raster_unit(int i, int tiles_m, int tiles_n, int ksp, int g) {
    const int per_group = g * tiles_n * ksp;
    const int G = i / per_group, rem = i - G * per_group;
    const int tm0 = G * g;
    const int gh = min(g, tiles_m - tm0);
    const int tn = rem / (gh * ksp);
    const int r2 = rem - tn * gh * ksp;
    const int tm = tm0 + r2 / ksp, ks = r2 % ksp;
    return (tm * tiles_n + tn) * ksp + ks;
}

// die_compact rule: every raster group is cut in two, die 0 first; after x units of the raster die 0
// holds floor(x * q0 / n_units) of them.
__device__ inline int band_die(int i, int n_units, int q0, int group_len) {
    const int start = (i / group_len) * group_len;
    const int end = min(n_units, start + group_len);
    const int cut = (int)(((long long)end * q0) / n_units - ((long long)start * q0) / n_units);
    return (i - start) < cut ? 0 : 1;
}

__device__ inline bool avoided(const PolicyDev& p, int s) { return (p.avoid[s >> 6] >> (s & 63)) & 1ull; }

// ---- steps 2, 3, 4 and the header: one thread -------------------------------------------------
__global__ void k_select_sms(const ag_topo_map* __restrict__ topo, PolicyDev pol, int b, int n_units,
                             int tiles_m, int tiles_n, int32_t* __restrict__ image, PlanLayout lay) {
    // the chip's per-SM arrays go to shared memory first (one thread walking them in global memory costs milliseconds)
    __shared__ short s_die[AG_MAX_SM], s_gpc[AG_MAX_SM], s_tpc[AG_MAX_SM];
    __shared__ unsigned char s_rand[AG_MAX_SM];
    for (int s = threadIdx.x; s < topo->n_sm; s += blockDim.x) {
        s_rand[s] = topo->is_random[s];
        s_die[s] = (short)topo->die[s];
        s_gpc[s] = (short)topo->gpc[s];
        s_tpc[s] = (short)topo->tpc[s];
    }
    __syncthreads();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    __shared__ int cand[AG_MAX_SM];
    __shared__ int S[AG_MAX_SM];
    __shared__ short key_tpc[AG_MAX_GPC + 1][AG_MAX_SM / 2];
    __shared__ int key_nt[AG_MAX_GPC + 1];
    const int n_sm = topo->n_sm;
    int nc = 0;
    for (int s = 0; s < n_sm; ++s)
        if (!avoided(pol, s)) cand[nc++] = s;
    int ns = 0;
    if (pol.kind == AG_OBLIVIOUS) {
        if (pol.seed != 0) {
            const unsigned long long base = mix64(pol.seed);
            for (int i = nc - 1; i >= 1; --i) {
                const int j = (int)(mix64(base + (unsigned long long)i) % (unsigned long long)(i + 1));
                const int t = cand[i];
                cand[i] = cand[j];
                cand[j] = t;
            }
        }
        for (int i = 0; i < b; ++i) S[ns++] = cand[i];
    } else {
        int cnt[2] = {0, 0};
        for (int i = 0; i < nc; ++i) cnt[s_die[cand[i]] & 1]++;
        int primary = (pol.preferred_die == 0 || pol.preferred_die == 1) ? pol.preferred_die
                                                                           : (cnt[0] >= cnt[1] ? 0 : 1);
        const int n_gpc = topo->n_gpc;
        const int n_pass = pol.sm_select == 1 ? 1 : 2;  // GPC spread: both dies in one round-robin
        if (pol.cluster_size > 2) {
            // Sets for kernels that launch clusters of c blocks: whole blocks of c normal SMs per GPC, dealt round-robin
            // over the GPCs; then the normal SMs not yet taken, last the random and unplaced ones (Sections 5.1.1, 7.3).
            const int c = pol.cluster_size;
            __shared__ unsigned char taken[AG_MAX_SM];
            for (int s = 0; s < n_sm; ++s) taken[s] = 0;
            for (int pass_d = 0; pass_d < n_pass; ++pass_d) {
                const int d = pol.sm_select == 1 ? -1 : (pass_d == 0 ? primary : 1 - primary);
                bool any = true;
                for (int p = 0; any; ++p) {
                    any = false;
                    for (int key = 0; key < n_gpc; ++key) {
                        // block p of this GPC: its normal candidates number p*c .. p*c + c - 1 in ascending id
                        int seen = 0, first_i = -1, last_i = -1;
                        for (int i = 0; i < nc; ++i) {
                            const int s = cand[i];
                            if ((d >= 0 && s_die[s] != d) || s_rand[s] || s_gpc[s] != key) continue;
                            if (seen == p * c) first_i = i;
                            if (seen == p * c + c - 1) { last_i = i; break; }
                            ++seen;
                        }
                        if (last_i < 0) continue;          // fewer than (p + 1) * c normal SMs here
                        any = true;
                        if (ns + c > b) continue;          // a whole block no longer fits in the budget
                        for (int i = first_i; i <= last_i; ++i) {
                            const int s = cand[i];
                            if ((d >= 0 && s_die[s] != d) || s_rand[s] || s_gpc[s] != key) continue;
                            S[ns++] = s;
                            taken[s] = 1;
                        }
                    }
                }
            }
            for (int want_normal = 1; want_normal >= 0; --want_normal)
                for (int pass_d = 0; pass_d < n_pass; ++pass_d) {
                    const int d = pol.sm_select == 1 ? -1 : (pass_d == 0 ? primary : 1 - primary);
                    for (int i = 0; i < nc && ns < b; ++i) {
                        const int s = cand[i];
                        const int normal = (!s_rand[s] && s_gpc[s] >= 0) ? 1 : 0;
                        if (taken[s] || (d >= 0 && s_die[s] != d) || normal != want_normal) continue;
                        S[ns++] = s;
                        taken[s] = 1;
                    }
                }
        }
        for (int pass_d = 0; pass_d < n_pass && ns < b; ++pass_d) {
            const int d = pol.sm_select == 1 ? -1 : (pass_d == 0 ? primary : 1 - primary);
            // distinct TPC ids of the candidates of every GPC key (unplaced SMs: key n_gpc), ascending, built once
            for (int key = 0; key <= n_gpc; ++key) key_nt[key] = 0;
            for (int i = 0; i < nc; ++i) {
                const int s = cand[i];
                if (d >= 0 && s_die[s] != d) continue;
                const int key = s_gpc[s] >= 0 ? s_gpc[s] : n_gpc;
                const int t = s_tpc[s];
                short* lst = key_tpc[key];
                int nt = key_nt[key], pos = 0;
                bool dup = false;
                for (; pos < nt; ++pos) {
                    if (lst[pos] == t) { dup = true; break; }
                    if (lst[pos] > t) break;
                }
                if (dup) continue;
                for (int m = nt; m > pos; --m) lst[m] = lst[m - 1];
                lst[pos] = (short)t;
                key_nt[key] = nt + 1;
            }
            for (int p = 0; ns < b; ++p) {
                bool any = false;
                for (int key = 0; key <= n_gpc && ns < b; ++key) {
                    if (p >= key_nt[key]) continue;
                    any = true;
                    const int t = key_tpc[key][p];
                    for (int i = 0; i < nc && ns < b; ++i) {
                        const int s = cand[i];
                        if ((d < 0 || s_die[s] == d) && s_tpc[s] == t &&
                            (s_gpc[s] >= 0 ? s_gpc[s] : n_gpc) == key)
                            S[ns++] = s;
                    }
                }
                if (!any) break;
            }
        }
    }
    // ascending order
    for (int i = 1; i < ns; ++i) {
        const int v = S[i];
        int j = i - 1;
        while (j >= 0 && S[j] > v) { S[j + 1] = S[j]; --j; }
        S[j + 1] = v;
    }
    int n_d[2] = {0, 0};
    for (int s = 0; s < n_sm; ++s) image[lay.smid_to_slot() + s] = -1;
    for (int i = 0; i < ns; ++i) {
        const int d = s_die[S[i]] & 1;
        image[lay.sm_list() + i] = S[i];
        image[lay.sm_die() + i] = d;
        image[lay.rank_in_die() + i] = n_d[d]++;
        image[lay.smid_to_slot() + S[i]] = i;
    }
    image[lay.die_sm_count() + 0] = n_d[0];
    image[lay.die_sm_count() + 1] = n_d[1];
    // quotas: floor share, leftovers by largest remainder (tie -> lower die)
    // (die_quota = 1: every die that holds SMs counts the same, whatever its SM count)
    long long q[2], rem[2];
    const int w_d[2] = {pol.die_quota ? (n_d[0] > 0) : n_d[0], pol.die_quota ? (n_d[1] > 0) : n_d[1]};
    const int w_all = w_d[0] + w_d[1];
    for (int d = 0; d < 2; ++d) {
        q[d] = (long long)n_units * w_d[d] / w_all;
        rem[d] = (long long)n_units * w_d[d] % w_all;
    }
    long long left = n_units - q[0] - q[1];
    const int first = rem[1] > rem[0] ? 1 : 0;
    for (int t = 0; t < 2 && left > 0; ++t) {
        const int d = t == 0 ? first : 1 - first;
        if (n_d[d] > 0) { q[d]++; left--; }
    }
    image[lay.die_q_off() + 0] = 0;
    image[lay.die_q_off() + 1] = (int)q[0];
    image[lay.die_q_off() + 2] = n_units;
    image[H_MAGIC] = kPlanMagic;
    image[H_KIND] = pol.kind;
    image[H_NSM] = n_sm;
    image[H_B] = b;
    image[H_NDIE] = 2;
    image[H_NUNITS] = n_units;
    image[H_TILES_M] = tiles_m;
    image[H_TILES_N] = tiles_n;
    image[H_KSPLITS] = pol.k_splits;
    image[H_TILE_M] = pol.tile_m;
    image[H_TILE_N] = pol.tile_n;
    image[H_M] = pol.M;
    image[H_N] = pol.N;
    image[H_K] = pol.K;
    image[H_STATIC] = pol.static_assign;
    image[H_ZERO] = 0;
}

// ---- step 5 (affinity): byte margins, one warp per raster index ---------------------------------
__device__ inline void add_interval(const uint8_t* __restrict__ doc, long long s, long long e, long long& l0,
                                    long long& l1) {
    while (s < e) {
        const long long c = s / AG_CHUNK_BYTES;
        const long long nxt = min(e, (c + 1) * (long long)AG_CHUNK_BYTES);
        if (doc[c]) l1 += nxt - s; else l0 += nxt - s;
        s = nxt;
    }
}

__global__ void k_score_units(PolicyDev pol, int n_units, int tiles_m, int tiles_n,
                              const uint8_t* __restrict__ doc, long long* __restrict__ margins) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= n_units) return;
    const int u = raster_unit(warp, tiles_m, tiles_n, pol.k_splits, pol.raster_group);
    const int ks = u % pol.k_splits, t = u / pol.k_splits;
    const int tm = t / tiles_n, tn = t % tiles_n;
    const int r0 = tm * pol.tile_m, r1 = min(pol.M, r0 + pol.tile_m);
    const int c0 = tn * pol.tile_n, c1 = min(pol.N, c0 + pol.tile_n);
    const int n_slab = (pol.K + pol.k_unit - 1) / pol.k_unit;
    const int per = (n_slab + pol.k_splits - 1) / pol.k_splits;
    const int k0 = min(pol.K, min(n_slab, ks * per) * pol.k_unit);
    const int k1 = min(pol.K, min(n_slab, (ks + 1) * per) * pol.k_unit);
    long long l0 = 0, l1 = 0;
    if (pol.a.present)
        for (int r = r0 + lane; r < r1; r += 32) {
            const long long base = pol.a.offset + (long long)r * pol.a.row_stride;
            add_interval(doc, base + (long long)k0 * pol.a.elem_bytes, base + (long long)k1 * pol.a.elem_bytes, l0, l1);
        }
    if (pol.b.present) {
        if (pol.b.layout == AG_LAYOUT_PAGED) {
            // 4 KB pages of [128 columns x 16 k]; a unit column holds tile_n / 128 column blocks
            const int ppt = (pol.K + 15) / 16;
            const int ppc = max(1, pol.tile_n / 128);
            for (int pc = tn * ppc; pc < (tn + 1) * ppc; ++pc)
                for (int k16 = k0 / 16 + lane; k16 < (k1 + 15) / 16; k16 += 32) {
                    const int phys = pol.b.page_table[(long long)pc * ppt + k16];
                    if (doc[phys]) l1 += AG_CHUNK_BYTES; else l0 += AG_CHUNK_BYTES;
                }
        } else {
            for (int k = k0 + lane; k < k1; k += 32) {
                const long long base = pol.b.offset + (long long)k * pol.b.row_stride;
                add_interval(doc, base + (long long)c0 * pol.b.elem_bytes, base + (long long)c1 * pol.b.elem_bytes, l0, l1);
            }
        }
    }
    if (pol.c.present)
        for (int r = r0 + lane; r < r1; r += 32) {
            const long long base = pol.c.offset + (long long)r * pol.c.row_stride;
            add_interval(doc, base + (long long)c0 * pol.c.elem_bytes, base + (long long)c1 * pol.c.elem_bytes, l0, l1);
        }
    long long m = l0 - l1;
    for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
    if (lane == 0) margins[warp] = m;
}

// Block-wide helpers for k_assign (called by every thread of the block, blockDim.x a multiple of 32, at most 1024).
__device__ inline int block_sum(int v, int* s_warp) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                       // s_warp may still be read by the call before
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = 0;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) t += s_warp[k];
    return t;
}
// number of set flags at lower thread ids; total = set flags of the whole block
__device__ inline int block_excl_scan_flag(bool f, int* s_warp, int& total) {
    const unsigned m = __ballot_sync(0xffffffffu, f);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) s_warp[w] = __popc(m);
    __syncthreads();
    int before = 0, t = 0;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) {
        const int c = s_warp[k];
        before += k < w ? c : 0;
        t += c;
    }
    total = t;
    return before + __popc(m & ((1u << lane) - 1u));
}

// ---- steps 5-6: unit -> die, per-die queues, per-SM lists: one thread block ----------------------
__global__ void __launch_bounds__(1024)
k_assign(PolicyDev pol, int b, int n_units, int tiles_m, int tiles_n, const long long* __restrict__ margins,
         int32_t* __restrict__ image, PlanLayout lay, int32_t* __restrict__ die_of) {
    const int tid = threadIdx.x, nt = blockDim.x;
    __shared__ int n_d[2];
    __shared__ int slots_of_die[2][AG_MAX_SM];
    __shared__ int s_warp[32];
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_sel[2];     // radix select: key prefix found so far, rank still to go
    if (tid == 0) {
        s_sel[0] = 0;
        n_d[0] = image[lay.die_sm_count()];
        n_d[1] = image[lay.die_sm_count() + 1];
        int c[2] = {0, 0};
        for (int i = 0; i < b; ++i) {
            const int d = image[lay.sm_die() + i];
            slots_of_die[d][c[d]++] = i;
        }
    }
    __syncthreads();
    const int q0 = image[lay.die_q_off() + 1];
    const int q[2] = {q0, n_units - q0};
    const int group_len = pol.raster_group * tiles_n * pol.k_splits;

    if (pol.kind == AG_OBLIVIOUS) {
        for (int i = tid; i < n_units; i += nt) {
            const int P = b / 2;
            const int slot = (pol.pair_lists && P > 0) ? 2 * (i % P) + ((i / P) & 1) : i % b;
            die_of[i] = image[lay.sm_die() + slot];
        }
    } else if (pol.kind == AG_DIE_COMPACT) {
        for (int i = tid; i < n_units; i += nt) die_of[i] = band_die(i, n_units, q0, group_len);
    } else {
        // The greedy pass of the plan (units in the order |margin| descending, raster index ascending; a unit takes the
        // die it prefers while that die has quota left, else the other) in closed form.  Until a die is full every unit
        // gets its preference, and once a die is full everything goes to the other one; the quotas add up to the unit
        // count, so at most one die d has more takers than quota q[d], and it keeps exactly its first q[d] takers in
        // that order.  Their cut is found by a radix select over the 64-bit keys (eight histogram passes) and a prefix
        // count over the units that tie with the cut; no sort, any unit count.
        auto key_pref = [&](int i, int& pref) -> unsigned long long {
            long long m = margins[i];
            if (pol.invert) m = -m;
            long long am = m < 0 ? -m : m;
            if (am < pol.min_margin) { am = 0; m = 0; }
            pref = m > 0 ? 0 : (m < 0 ? 1 : band_die(i, n_units, q0, group_len));
            return (unsigned long long)am;
        };
        int mine0 = 0;
        for (int i = tid; i < n_units; i += nt) {
            int pref;
            key_pref(i, pref);
            mine0 += pref == 0;
        }
        const int n_pref0 = block_sum(mine0, s_warp);
        const int d_full = n_pref0 > q[0] ? 0 : ((n_units - n_pref0) > q[1] ? 1 : -1);
        unsigned long long cut = 0;    // key of the last taker that die d_full keeps
        int keep_ties = 0;             // how many takers with exactly that key it keeps (lowest raster indices)
        if (d_full >= 0 && q[d_full] > 0) {
            if (tid == 0) {
                s_sel[0] = 0;
                s_sel[1] = (unsigned long long)q[d_full];
            }
            __syncthreads();
            for (int byte = 7; byte >= 0; --byte) {
                for (int k = tid; k < 256; k += nt) hist[k] = 0;
                __syncthreads();
                const unsigned long long prefix = s_sel[0];
                for (int i = tid; i < n_units; i += nt) {
                    int pref;
                    const unsigned long long key = key_pref(i, pref);
                    if (pref == d_full && (byte == 7 || (key >> (8 * (byte + 1))) == prefix))
                        atomicAdd(&hist[(unsigned)(key >> (8 * byte)) & 255u], 1u);
                }
                __syncthreads();
                if (tid == 0) {
                    unsigned long long rank = s_sel[1];     // 1-based rank of the cut among the keys that share the prefix
                    int bin = 255;
                    for (; bin > 0 && hist[bin] < rank; --bin) rank -= hist[bin];
                    s_sel[0] = (prefix << 8) | (unsigned long long)bin;
                    s_sel[1] = rank;
                }
                __syncthreads();
            }
            cut = s_sel[0];
            keep_ties = (int)s_sel[1];
        }
        int ties_before = 0;           // takers of d_full with key == cut at raster indices below the current chunk
        for (int base = 0; base < n_units; base += nt) {
            const int i = base + tid;
            int pref = 0;
            unsigned long long key = 0;
            if (i < n_units) key = key_pref(i, pref);
            const bool tie = i < n_units && d_full >= 0 && pref == d_full && key == cut;
            int total;
            const int pos = ties_before + block_excl_scan_flag(tie, s_warp, total);
            ties_before += total;
            if (i < n_units) {
                int d = pref;
                if (pref == d_full && (q[d_full] == 0 || key < cut || (key == cut && pos >= keep_ties))) d = 1 - d_full;
                die_of[i] = d;
            }
        }
    }
    __syncthreads();
    // per-die queues in raster order: a unit's place is the number of units of its die before it
    int mine = 0;
    for (int i = tid; i < n_units; i += nt) mine += die_of[i] == 0;
    const int cnt0 = block_sum(mine, s_warp);
    const int cnt[2] = {cnt0, n_units - cnt0};
    int zeros_before = 0;
    for (int base = 0; base < n_units; base += nt) {
        const int i = base + tid;
        const bool z = i < n_units && die_of[i] == 0;
        int total;
        const int zb = zeros_before + block_excl_scan_flag(z, s_warp, total);
        zeros_before += total;
        if (i < n_units) {
            const int u = raster_unit(i, tiles_m, tiles_n, pol.k_splits, pol.raster_group);
            image[lay.die_q() + (z ? zb : cnt0 + (i - zb))] = u;
        }
    }
    if (tid == 0) {
        image[lay.die_q_off() + 0] = 0;
        image[lay.die_q_off() + 1] = cnt[0];
        image[lay.die_q_off() + 2] = n_units;
        // list lengths and offsets
        int off = 0;
        for (int s = 0; s < b; ++s) {
            image[lay.sm_q_off() + s] = off;
            int len;
            if (pol.pair_lists) {
                // entries are dealt to TPCs: entry i -> TPC (i mod P), its lower SM when (i div P) is even
                const int d = image[lay.sm_die() + s];
                const int r = pol.kind == AG_OBLIVIOUS ? s : image[lay.rank_in_die() + s];
                const int total = pol.kind == AG_OBLIVIOUS ? n_units : cnt[d];
                const int P = (pol.kind == AG_OBLIVIOUS ? b : n_d[d]) / 2;
                const int j = r >> 1, par = r & 1;
                const int T = (P > 0 && j < P && total > j) ? (total - j + P - 1) / P : 0;  // rounds in which TPC j gets a unit
                len = par ? T / 2 : (T + 1) / 2;
            } else if (pol.kind == AG_OBLIVIOUS) {
                len = n_units > s ? (n_units - s + b - 1) / b : 0;
            } else {
                const int d = image[lay.sm_die() + s], r = image[lay.rank_in_die() + s];
                len = cnt[d] > r ? (cnt[d] - r + n_d[d] - 1) / n_d[d] : 0;
            }
            off += len;
        }
        image[lay.sm_q_off() + b] = off;
    }
    __syncthreads();
    if (pol.kind == AG_OBLIVIOUS) {
        const int P = b / 2;
        for (int i = tid; i < n_units; i += nt) {
            const int u = raster_unit(i, tiles_m, tiles_n, pol.k_splits, pol.raster_group);
            if (pol.pair_lists && P > 0) {
                const int t = i / P;
                image[lay.sm_q() + image[lay.sm_q_off() + 2 * (i % P) + (t & 1)] + t / 2] = u;
            } else {
                image[lay.sm_q() + image[lay.sm_q_off() + (i % b)] + i / b] = u;
            }
        }
    } else {
        const int len0 = image[lay.die_q_off() + 1];
        for (int e = tid; e < n_units; e += nt) {
            const int d = e < len0 ? 0 : 1;
            const int idx = d == 0 ? e : e - len0;
            const int P = n_d[d] / 2;
            if (pol.pair_lists && P > 0) {
                const int t = idx / P;
                const int slot = slots_of_die[d][2 * (idx % P) + (t & 1)];
                image[lay.sm_q() + image[lay.sm_q_off() + slot] + t / 2] = image[lay.die_q() + e];
            } else {
                const int slot = slots_of_die[d][idx % n_d[d]];
                image[lay.sm_q() + image[lay.sm_q_off() + slot] + idx / n_d[d]] = image[lay.die_q() + e];
            }
        }
    }
}

}  // namespace ag

using namespace ag;

static OperandDev to_dev(const ag_operand_desc& o, const int32_t* d_table) {
    OperandDev r;
    r.present = o.present;
    r.layout = o.layout;
    r.elem_bytes = o.elem_bytes;
    r.pad = 0;
    r.offset = o.offset;
    r.row_stride = o.row_stride;
    r.page_table = d_table;
    return r;
}

static bool operand_in_range(const ag_operand_desc& o, long long rows, long long cols, size_t bytes) {
    if (!o.present) return true;
    if (o.layout == AG_LAYOUT_PAGED) return o.page_table != nullptr && o.n_pages > 0;
    if (o.elem_bytes <= 0 || o.offset < 0 || o.row_stride < cols * o.elem_bytes) return false;
    const long long last = o.offset + (rows - 1) * o.row_stride + cols * o.elem_bytes;
    return (size_t)last <= bytes;
}

extern "C" ag_status sched_build(const ag_topo_map* map, const ag_affinity_map* amap, int sm_budget,
                                 const ag_policy* policy, ag_plan** out) {
    if (!map || !policy || !out) return AG_ERR_ARG;
    *out = nullptr;
    const ag_policy& p = *policy;
    if (map->n_sm <= 0 || map->n_sm > AG_MAX_SM) return AG_ERR_ARG;
    if (p.kind < AG_OBLIVIOUS || p.kind > AG_AFFINITY) return AG_ERR_ARG;
    if (p.M <= 0 || p.N <= 0 || p.K <= 0 || p.tile_m <= 0 || p.tile_n <= 0) return AG_ERR_ARG;
    if (p.k_splits < 1 || p.k_unit < 1 || p.raster_group < 1 || p.min_margin < 0) return AG_ERR_ARG;
    if (p.sm_select < 0 || p.sm_select > 1) return AG_ERR_ARG;
    if (p.cluster_size != 0 && p.cluster_size != 1 && p.cluster_size != 2 && p.cluster_size != 4 && p.cluster_size != 8) return AG_ERR_ARG;
    if (p.kind == AG_AFFINITY && !amap) return AG_ERR_ARG;
    int n_cand = 0;
    for (int s = 0; s < map->n_sm; ++s)
        if (!((p.avoid_sm_mask[s >> 6] >> (s & 63)) & 1ull)) ++n_cand;
    if (sm_budget < 1 || sm_budget > n_cand) return AG_ERR_ARG;
    const int n_slab = (p.K + p.k_unit - 1) / p.k_unit;
    const int per = (n_slab + p.k_splits - 1) / p.k_splits;
    if ((long long)(p.k_splits - 1) * per >= n_slab) return AG_ERR_ARG;  // an empty k-split
    const long long tiles_m = (p.M + p.tile_m - 1) / p.tile_m, tiles_n = (p.N + p.tile_n - 1) / p.tile_n;
    const long long n_units_ll = tiles_m * tiles_n * p.k_splits;
    if (n_units_ll > (1 << 20)) return AG_ERR_ARG;
    const int n_units = (int)n_units_ll;
    if (p.kind == AG_AFFINITY) {
        if (!operand_in_range(p.a, p.M, p.K, amap->bytes) || !operand_in_range(p.c, p.M, p.N, amap->bytes))
            return AG_ERR_ARG;
        if (!operand_in_range(p.b, p.K, p.N, amap->bytes)) return AG_ERR_ARG;
        if (p.b.present && p.b.layout == AG_LAYOUT_PAGED) {
            const long long need = tiles_n * (p.tile_n >= 128 ? p.tile_n / 128 : 1) * ((p.K + 15) / 16);
            if (p.b.n_pages < need) return AG_ERR_ARG;
            for (long long i = 0; i < need; ++i)
                if (p.b.page_table[i] < 0 || (size_t)p.b.page_table[i] >= amap->n_chunks) return AG_ERR_ARG;
        }
        if ((p.a.present && p.a.layout != AG_LAYOUT_ROWMAJOR) || (p.c.present && p.c.layout != AG_LAYOUT_ROWMAJOR))
            return AG_ERR_ARG;
    }
    int dev = 0;
    AG_CUDA(cudaGetDevice(&dev));

    ag_plan* pl = new (std::nothrow) ag_plan();
    if (!pl) return AG_ERR_NOMEM;
    pl->lay = PlanLayout{sm_budget, n_units, map->n_sm};
    pl->policy = p;
    pl->policy.a.page_table = pl->policy.b.page_table = pl->policy.c.page_table = nullptr;
    pl->d_image = nullptr; pl->d_ctrl = nullptr; pl->d_tile_owner = nullptr; pl->d_tile_count = nullptr;
    pl->d_margins = nullptr;
    pl->d_unit_times = nullptr;
    pl->d_partial = nullptr; pl->d_quick = nullptr;
    pl->epoch = 0;
    pl->grid_blocks = 0;
    pl->kslabs_total = n_slab;
    pl->kslabs_per_split = per;
    pl->tm_a_ptr = pl->tm_b_ptr = nullptr; pl->tm_c_ptr = nullptr;

    ag_topo_map* d_topo = nullptr;
    int32_t* d_table = nullptr;
    int32_t* d_die_of = nullptr;
    ag_status st = AG_OK;
    auto fail = [&](cudaError_t e) { st = cuda_fail(e); };
    cudaError_t e;
#define TRY(x) do { e = (x); if (e != cudaSuccess) { fail(e); goto done; } } while (0)
    {
        const size_t image_bytes = sizeof(int32_t) * (size_t)pl->lay.total();
        TRY(cudaMalloc(&pl->d_image, image_bytes));
        TRY(cudaMalloc(&pl->d_ctrl, sizeof(PlanCtrl)));
        TRY(cudaMemset(pl->d_ctrl, 0, sizeof(PlanCtrl)));
        TRY(cudaMalloc(&pl->d_tile_owner, sizeof(int32_t) * n_units));
        TRY(cudaMalloc(&pl->d_tile_count, sizeof(int32_t) * n_units));
        TRY(cudaMemset(pl->d_tile_owner, 0xFF, sizeof(int32_t) * n_units));
        TRY(cudaMemset(pl->d_tile_count, 0, sizeof(int32_t) * n_units));
        if (p.tile_n == 128 && (p.tile_m <= 64 || (p.tile_m == 128 && p.decode_shaped)) && p.k_splits > 1 && !p.splitk_in_memory) {
            // decode-shaped plans: split-K partial sums and per-tile arrival counters
            TRY(cudaMalloc(&pl->d_partial, sizeof(float) * (size_t)p.k_splits * p.M * p.N));
        }
        TRY(cudaMalloc(&d_topo, sizeof(ag_topo_map)));
        TRY(cudaMemcpy(d_topo, map, sizeof(ag_topo_map), cudaMemcpyHostToDevice));
        TRY(cudaMalloc(&d_die_of, sizeof(int32_t) * n_units));
        if (p.kind == AG_AFFINITY && p.b.present && p.b.layout == AG_LAYOUT_PAGED) {
            TRY(cudaMalloc(&d_table, sizeof(int32_t) * (size_t)p.b.n_pages));
            TRY(cudaMemcpy(d_table, p.b.page_table, sizeof(int32_t) * (size_t)p.b.n_pages, cudaMemcpyHostToDevice));
        }
        PolicyDev pd;
        memset(&pd, 0, sizeof pd);
        pd.kind = p.kind; pd.M = p.M; pd.N = p.N; pd.K = p.K; pd.tile_m = p.tile_m; pd.tile_n = p.tile_n;
        pd.k_splits = p.k_splits; pd.k_unit = p.k_unit; pd.raster_group = p.raster_group;
        pd.preferred_die = p.preferred_die; pd.invert = p.invert_affinity; pd.static_assign = p.static_assign;
        pd.seed = p.seed;
        pd.sm_select = p.sm_select;
        pd.cluster_size = p.cluster_size;
        pd.die_quota = p.die_quota ? 1 : 0;
        pd.pair_lists = p.pair_lists ? 1 : 0;
        pd.min_margin = p.min_margin;
        for (int i = 0; i < 4; ++i) pd.avoid[i] = p.avoid_sm_mask[i];
        pd.a = to_dev(p.a, nullptr); pd.b = to_dev(p.b, d_table); pd.c = to_dev(p.c, nullptr);

        k_select_sms<<<1, 32>>>(d_topo, pd, sm_budget, n_units, (int)tiles_m, (int)tiles_n, pl->d_image, pl->lay);
        count_launch();
        TRY(cudaGetLastError());
        if (p.kind == AG_AFFINITY) {
            TRY(cudaMalloc(&pl->d_margins, sizeof(long long) * n_units));
            const int warps_per_block = 8;
            const int blocks = (n_units + warps_per_block - 1) / warps_per_block;
            k_score_units<<<blocks, warps_per_block * 32>>>(pd, n_units, (int)tiles_m, (int)tiles_n,
                                                            amap->d_die_of_chunk, pl->d_margins);
            count_launch();
            TRY(cudaGetLastError());
        }
        k_assign<<<1, 1024>>>(pd, sm_budget, n_units, (int)tiles_m, (int)tiles_n, pl->d_margins, pl->d_image,
                              pl->lay, d_die_of);
        count_launch();
        TRY(cudaGetLastError());
        TRY(cudaDeviceSynchronize());
        pl->h_image.resize(pl->lay.total());
        TRY(cudaMemcpy(pl->h_image.data(), pl->d_image, image_bytes, cudaMemcpyDeviceToHost));
        memcpy(pl->header, pl->h_image.data(), sizeof pl->header);
        {
            // per SM id: its slot, its list and the list's first unit in one 16-byte entry, so that a block
            // learns all of it with a single load
            const int32_t* img = pl->h_image.data();
            std::vector<int4> quick(map->n_sm);
            for (int s = 0; s < map->n_sm; ++s) {
                const int slot = img[pl->lay.smid_to_slot() + s];
                int4 q = make_int4(-1, 0, 0, -1);
                if (slot >= 0) {
                    q.x = slot;
                    q.y = img[pl->lay.sm_q_off() + slot];
                    q.z = img[pl->lay.sm_q_off() + slot + 1] - q.y;
                    q.w = q.z > 0 ? img[pl->lay.sm_q() + q.y] : -1;
                }
                quick[s] = q;
            }
            TRY(cudaMalloc(&pl->d_quick, sizeof(int4) * map->n_sm));
            TRY(cudaMemcpy(pl->d_quick, quick.data(), sizeof(int4) * map->n_sm, cudaMemcpyHostToDevice));
        }
        if (p.pair_lists) {
            // units were dealt to TPCs: every chosen TPC must be whole (both SMs chosen, adjacent in the die's ranks)
            const int32_t* img = pl->h_image.data();
            const int groups = p.kind == AG_OBLIVIOUS ? 1 : 2;
            for (int d = 0; d < groups && st == AG_OK; ++d) {
                std::vector<int> sms;
                for (int i = 0; i < sm_budget; ++i)
                    if (groups == 1 || img[pl->lay.sm_die() + i] == d) sms.push_back(img[pl->lay.sm_list() + i]);
                if (sms.size() % 2) st = AG_ERR_ARG;
                for (size_t j = 0; j + 1 < sms.size() && st == AG_OK; j += 2)
                    if (map->tpc[sms[j]] != map->tpc[sms[j + 1]]) st = AG_ERR_ARG;
            }
        }
    }
done:
#undef TRY
    cudaFree(d_topo);
    cudaFree(d_table);
    cudaFree(d_die_of);
    if (st != AG_OK) {
        ag_plan_destroy(pl);
        return st;
    }
    *out = pl;
    return AG_OK;
}

extern "C" ag_status ag_plan_export(const ag_plan* plan, int32_t* outw, size_t cap, size_t* n_words) {
    if (!plan) return AG_ERR_ARG;
    if (n_words) *n_words = plan->h_image.size();
    if (!outw) return n_words ? AG_OK : AG_ERR_ARG;
    if (cap < plan->h_image.size()) return AG_ERR_ARG;
    memcpy(outw, plan->h_image.data(), plan->h_image.size() * sizeof(int32_t));
    return AG_OK;
}

extern "C" ag_status ag_plan_margins(const ag_plan* plan, int64_t* outm, size_t cap) {
    if (!plan || !outm || !plan->d_margins || cap < (size_t)plan->lay.n_units) return AG_ERR_ARG;
    AG_CUDA(cudaMemcpy(outm, plan->d_margins, sizeof(long long) * plan->lay.n_units, cudaMemcpyDeviceToHost));
    return AG_OK;
}

extern "C" ag_status ag_plan_tile_record(const ag_plan* plan, int32_t* owner_sm, int32_t* run_count, size_t cap) {
    if (!plan || cap < (size_t)plan->lay.n_units) return AG_ERR_ARG;
    if (owner_sm)
        AG_CUDA(cudaMemcpy(owner_sm, plan->d_tile_owner, sizeof(int32_t) * plan->lay.n_units, cudaMemcpyDeviceToHost));
    if (run_count)
        AG_CUDA(cudaMemcpy(run_count, plan->d_tile_count, sizeof(int32_t) * plan->lay.n_units, cudaMemcpyDeviceToHost));
    return AG_OK;
}

extern "C" ag_status ag_plan_reset_record(ag_plan* plan) {
    if (!plan) return AG_ERR_ARG;
    AG_CUDA(cudaMemset(plan->d_tile_owner, 0xFF, sizeof(int32_t) * plan->lay.n_units));
    AG_CUDA(cudaMemset(plan->d_tile_count, 0, sizeof(int32_t) * plan->lay.n_units));
    return AG_OK;
}

extern "C" ag_status ag_plan_trace(ag_plan* plan, int on) {
    if (!plan) return AG_ERR_ARG;
    if (on && !plan->d_unit_times) {
        AG_CUDA(cudaMalloc(&plan->d_unit_times, sizeof(unsigned long long) * 2 * plan->lay.n_units));
        AG_CUDA(cudaMemset(plan->d_unit_times, 0, sizeof(unsigned long long) * 2 * plan->lay.n_units));
    } else if (!on && plan->d_unit_times) {
        AG_CUDA(cudaDeviceSynchronize());
        cudaFree(plan->d_unit_times);
        plan->d_unit_times = nullptr;
    }
    return AG_OK;
}

extern "C" ag_status ag_plan_unit_times(const ag_plan* plan, uint64_t* start_ns, uint64_t* end_ns, size_t cap) {
    if (!plan || !plan->d_unit_times || !start_ns || !end_ns || cap < (size_t)plan->lay.n_units) return AG_ERR_ARG;
    std::vector<unsigned long long> t(2 * (size_t)plan->lay.n_units);
    AG_CUDA(cudaMemcpy(t.data(), plan->d_unit_times, sizeof(unsigned long long) * t.size(), cudaMemcpyDeviceToHost));
    for (int u = 0; u < plan->lay.n_units; ++u) {
        start_ns[u] = t[2 * (size_t)u];
        end_ns[u] = t[2 * (size_t)u + 1];
    }
    return AG_OK;
}

extern "C" ag_status ag_cluster_capacity(const ag_plan* plan, const ag_topo_map* map, int cluster_size, int32_t* n_clusters) {
    if (!plan || !map || !n_clusters || cluster_size < 1 || cluster_size > 16 || map->n_sm != plan->lay.n_sm) return AG_ERR_ARG;
    std::vector<int> per_gpc(AG_MAX_GPC, 0), loose_tpc(AG_MAX_SM, 0);
    int total = 0;
    const int32_t* list = plan->h_image.data() + plan->lay.sm_list();
    for (int i = 0; i < plan->lay.b; ++i) {
        const int s = list[i];
        const bool placed = map->gpc[s] >= 0 && map->gpc[s] < AG_MAX_GPC;
        if (cluster_size > 2 && (map->is_random[s] || !placed)) continue;
        if (placed) per_gpc[map->gpc[s]]++;
        else loose_tpc[(map->tpc[s] >= 0 && map->tpc[s] < AG_MAX_SM) ? map->tpc[s] : 0]++;   // an unplaced SM is only known to share a TPC with its neighbour
    }
    for (int g = 0; g < AG_MAX_GPC; ++g) total += per_gpc[g] / cluster_size;
    for (int t = 0; t < AG_MAX_SM; ++t) total += loose_tpc[t] / cluster_size;
    *n_clusters = total;
    return AG_OK;
}

extern "C" ag_status ag_plan_set_grid(ag_plan* plan, int blocks) {
    if (!plan || blocks < 0 || blocks > plan->lay.n_sm) return AG_ERR_ARG;
    plan->grid_blocks = blocks;
    return AG_OK;
}

extern "C" ag_status ag_plan_adopted(const ag_plan* plan, uint32_t* n_lists) {
    if (!plan || !n_lists) return AG_ERR_ARG;
    PlanCtrl c;
    AG_CUDA(cudaMemcpy(&c, plan->d_ctrl, sizeof(int) * 8, cudaMemcpyDeviceToHost));
    *n_lists = c.adopted;
    return AG_OK;
}

extern "C" ag_status ag_last_status(const ag_plan* plan) {
    if (!plan) return AG_ERR_ARG;
    PlanCtrl c;
    AG_CUDA(cudaMemcpy(&c, plan->d_ctrl, sizeof(int) * 8, cudaMemcpyDeviceToHost));
    if (c.status != 0) return (ag_status)c.status;
    if (plan->epoch != 0) {
        std::vector<unsigned int> claimed(plan->lay.b);
        AG_CUDA(cudaMemcpy(claimed.data(), (const char*)plan->d_ctrl + offsetof(PlanCtrl, claimed) + sizeof(unsigned int) * AG_MAX_SM * (plan->epoch & 1u),
                           sizeof(unsigned int) * plan->lay.b, cudaMemcpyDeviceToHost));
        int n_claimed = 0;
        for (int i = 0; i < plan->lay.b; ++i) n_claimed += claimed[i] == plan->epoch;
        // static lists: every list must have been run by somebody (its own SM's block or one that took it over);
        // dynamic queues: any block drains them, so one is enough
        if (plan->header[H_STATIC] ? n_claimed != plan->lay.b : n_claimed == 0) return AG_ERR_UNMANNED_SM;
    }
    return AG_OK;
}

extern "C" ag_status ag_last_status_where(const ag_plan* plan, int32_t* role, int32_t* smid) {
    if (!plan) return AG_ERR_ARG;
    PlanCtrl c;
    AG_CUDA(cudaMemcpy(&c, plan->d_ctrl, sizeof(int) * 8, cudaMemcpyDeviceToHost));
    if (role) *role = c.status != 0 ? (c.status_info >> 16) : 0;
    if (smid) *smid = c.status != 0 ? (c.status_info & 0xffff) : -1;
    return AG_OK;
}

extern "C" void ag_plan_destroy(ag_plan* plan) {
    if (!plan) return;
    cudaFree(plan->d_image);
    cudaFree(plan->d_ctrl);
    cudaFree(plan->d_tile_owner);
    cudaFree(plan->d_tile_count);
    cudaFree(plan->d_margins);
    cudaFree(plan->d_unit_times);
    cudaFree(plan->d_partial);
    cudaFree(plan->d_quick);
    delete plan;
}
