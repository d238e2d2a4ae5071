// topo_discover and affinity_probe: per-chip discovery of compute and memory asymmetry.
//
//   census           every SM reports %smid once (grid = #SMs, one block per SM)
//   cluster probing  Section 5.1.1: thread-block clusters of size 3..8 are co-scheduled on one
//                    GPC; SM ids seen together are merged (union-find); SMs never seen are "random"
//   latency probing  Section 6.1.1 + appendix (HBM latency kernel): single thread, invalidate the
//                    L2 line, L1-bypassing load, SM cycle counter; run from every SM it splits
//                    the SMs into two partitions (dies)
//   bandwidth probe  Section 5.1.2: SMs of one GPC share its crossbar port to L2; a random TPC
//                    belongs to the GPC whose known SMs it slows down
//   affinity probe   Section 6.1: chunk -> die from the two latency tiers, 4 KB chunks
//
// Pinning: a kernel cannot choose its SMs, so every probe launches one block per SM and lets
// the blocks that landed on the wanted SMs work.  The others stay resident (bounded) until the
// wanted SMs have checked in, so that all blocks sit on distinct SMs.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <numeric>
#include <vector>

#include "internal.h"
#include "ptx.cuh"

namespace ag {

constexpr int kPinSmem = 120 * 1024;  // > half of an SM's shared memory: at most one block per SM
constexpr int kRefChunks = 64;        // reference chunks for the SM -> die probe
constexpr int kLatReps = 8;           // min over this many timed loads

struct PinCtrl {
    unsigned int arrived;   // members that have checked in
    unsigned int pad[3];
    unsigned long long t_start[AG_MAX_SM];
    unsigned long long t_end[AG_MAX_SM];
};

// Members check in; everybody then waits (at most wait_ns) until all members are there.
__device__ inline void pin_rendezvous(PinCtrl* pc, bool member, unsigned int n_members, unsigned long long wait_ns) {
    if (threadIdx.x == 0) {
        if (member) atomicAdd(&pc->arrived, 1u);
        const unsigned long long t0 = globaltimer_ns();
        while (*reinterpret_cast<volatile unsigned int*>(&pc->arrived) < n_members) {
            if (globaltimer_ns() - t0 > wait_ns) break;
            __nanosleep(100);
        }
    }
    __syncthreads();
}

__device__ __forceinline__ unsigned long long clock64_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t)::"memory");
    return t;
}

// One timed L1-bypassing load; the add that consumes the value sits between the load and the
// second clock read, so the clock is read only after the data has arrived.
__device__ __forceinline__ uint32_t timed_load_cg(const void* p, uint32_t& sink) {
    const unsigned long long t0 = clock64_now();
    uint32_t v = ld_cg_u32(p);
    asm volatile("add.u32 %0, %0, %1;" : "+r"(sink) : "r"(v) : "memory");
    const unsigned long long t1 = clock64_now();
    return (uint32_t)(t1 - t0);
}

// ---- census ---------------------------------------------------------------------------------
__global__ void k_census(PinCtrl* pc, int* count, unsigned int n_blocks) {
    if (threadIdx.x == 0) atomicAdd(&count[smid()], 1);
    pin_rendezvous(pc, true, n_blocks, 100000ull);
}

// ---- cluster probe ---------------------------------------------------------------------------
__global__ void k_cluster_probe(int* smid_of_block) {
    if (threadIdx.x == 0) {
        smid_of_block[blockIdx.x] = (int)smid();
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 20000ull) __nanosleep(500);  // stay a while so clusters spread out
    }
}

// Cluster layout: every block notes its SM and start time, then stays until all blocks of the launch have started
// (or 50 us have passed), so that one launch shows which SMs the hardware groups into clusters when all are wanted.
__global__ void k_cluster_layout(int* smid_of_block, unsigned long long* start_ns, unsigned int* started, unsigned int n_blocks) {
    if (threadIdx.x == 0) {
        smid_of_block[blockIdx.x] = (int)smid();
        const unsigned long long t0 = globaltimer_ns();
        start_ns[blockIdx.x] = t0;
        atomicAdd(started, 1u);
        while (*reinterpret_cast<volatile unsigned int*>(started) < n_blocks && globaltimer_ns() - t0 < 50000ull) __nanosleep(500);
    }
}

// ---- latency probe from one SM -------------------------------------------------------------
// mode 0: save the line, invalidate it in L2 (discard.global.L2), timed load, write it back -
//         the HBM-latency kernel of the paper's appendix.
// mode 1: plain timed load (latency of whichever level holds the line).
// mode 2: rewrite the line with its own contents, then timed load.  The write leaves the line in
//         its home L2 partition and drops any copy replicated into the other partition, so the
//         load is an L2 hit in the home partition: short from a same-die SM, long across dies.
// out[r] = min over reps; raw (optional) keeps every sample.
__global__ void k_latency_from_sm(PinCtrl* pc, int target_sm, uint8_t* buf, const long long* line_off, int n_lines,
                                  int reps, int mode, uint32_t* out, uint32_t* raw /* n_lines x reps or null */) {
    const bool member = ((int)smid() == target_sm);
    pin_rendezvous(pc, member, 1, 100000ull);
    if (!member || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    uint32_t sink = 0;
    for (int r = 0; r < n_lines; ++r) {
        uint8_t* line = buf + line_off[r];
        uint32_t best = 0xffffffffu;
        for (int k = 0; k < reps; ++k) {
            uint32_t saved = 0;
            if (mode == 0 || mode == 2) {
                saved = ld_cg_u32(line + lane * 4);
                __syncwarp();
                if (mode == 2) {
                    reinterpret_cast<volatile uint32_t*>(line)[lane] = saved;
                    __threadfence();
                } else if (lane == 0) {
                    discard_l2_128(line);
                }
                __syncwarp();
            }
            if (lane == 0) {
                sink += ld_cg_u32(line + 256);  // another line of the same chunk: warms the address translation
                const uint32_t dt = timed_load_cg(line, sink);
                best = min(best, dt);
                if (raw) raw[r * reps + k] = dt;
            }
            __syncwarp();
            if (mode == 0) {
                reinterpret_cast<uint32_t*>(line)[lane] = saved;
                __threadfence();
            }
        }
        if (lane == 0) out[r] = best;
    }
    if (lane == 0 && sink == 0x12345678u) out[0] = sink;  // keep the loads alive
}

// ---- L2 bandwidth of a set of SMs ----------------------------------------------------------------
// 1024 threads, eight independent 16-byte loads in flight per thread, so that the SM's own
// request rate - not the load latency - is what the GPC's port to L2 has to carry.
__global__ void __launch_bounds__(1024)
k_l2_bandwidth(PinCtrl* pc, const unsigned long long* member_mask, unsigned int n_members, const uint4* buf,
               size_t slice_vec, int passes, unsigned int* sink_out) {
    const int sm = (int)smid();
    const bool member = (member_mask[sm >> 6] >> (sm & 63)) & 1ull;
    pin_rendezvous(pc, member, n_members, 200000ull);
    if (!member) return;
    // each member streams its own slice (warm-up pass untimed, then `passes` timed passes)
    const uint4* slice = buf + (size_t)(sm % 64) * slice_vec;
    unsigned int acc = 0;
    for (size_t i = threadIdx.x; i < slice_vec; i += blockDim.x) acc += ld_cg_u128(slice + i).x;
    __syncthreads();
    unsigned long long t0 = 0;
    if (threadIdx.x == 0) t0 = globaltimer_ns();
    const size_t step = (size_t)blockDim.x * 8;
    for (int p = 0; p < passes; ++p)
        for (size_t i0 = threadIdx.x; i0 + 7 * blockDim.x < slice_vec; i0 += step) {
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = ld_cg_u128(slice + i0 + (size_t)j * blockDim.x);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc += v[j].x ^ v[j].w;
        }
    __syncthreads();
    if (threadIdx.x == 0) {
        pc->t_start[sm] = t0;
        pc->t_end[sm] = globaltimer_ns();
    }
    if (acc == 0x9e3779b9u) sink_out[0] = acc;
}

// Keeps every SM busy for `ns` so that clocks have settled before cycle counts are compared.
__global__ void k_warm_up(unsigned long long ns, float* out) {
    const unsigned long long t0 = globaltimer_ns();
    float x = threadIdx.x * 1e-3f;
    while (globaltimer_ns() - t0 < ns) {
#pragma unroll
        for (int i = 0; i < 64; ++i) x = fmaf(x, 1.0001f, 0.5f);
    }
    if (x == 123.456f) out[0] = x;
}

// ---- bandwidth of one die's SMs over the chunks of one die (Section 6.2.1) ---------------------------------
// Members (the SMs of the reading die) split the listed chunks round-robin; every warp of a member streams whole
// chunks with eight independent 16-byte L1-bypassing loads per lane (8 warps x 4 KB in flight per SM).
__global__ void __launch_bounds__(256)
k_die_bandwidth(PinCtrl* pc, const int* member_rank, unsigned int n_members, const uint8_t* buf,
                const uint32_t* chunk_list, size_t n_list, int passes, unsigned int* sink_out) {
    const int sm = (int)smid();
    const int rank = member_rank[sm];
    pin_rendezvous(pc, rank >= 0, n_members, 200000ull);
    if (rank < 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    const size_t stride = (size_t)n_members * n_warps;
    unsigned int acc = 0;
    unsigned long long t0 = 0;
    __syncthreads();
    if (threadIdx.x == 0) t0 = globaltimer_ns();
    for (int p = 0; p < passes; ++p) {
        size_t i = (size_t)rank * n_warps + warp;
        uint32_t next = i < n_list ? chunk_list[i] : 0;
        for (; i < n_list; i += stride) {
            const uint4* chunk = reinterpret_cast<const uint4*>(buf + (size_t)next * AG_CHUNK_BYTES);
            if (i + stride < n_list) next = chunk_list[i + stride];   // index of the following chunk: off the critical path
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = ld_cg_u128(chunk + j * 32 + lane);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc += v[j].x ^ v[j].w;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        pc->t_start[sm] = t0;
        pc->t_end[sm] = globaltimer_ns();
    }
    if (acc == 0x9e3779b9u) sink_out[0] = acc;
}

// ---- affinity probe over a buffer -----------------------------------------------------------------
// Members (the SMs of one die) split the chunks round-robin; one warp per SM.  Per chunk: a few
// 128-byte lines, each saved, invalidated in L2, loaded with a timed L1-bypassing load, restored.
// With `list` (n_work chunk indices) only those chunks are probed and cycles[i] belongs to list[i]; without it
// all n_work chunks of the buffer are probed and cycles[c] belongs to chunk c.
__global__ void k_affinity_probe(PinCtrl* pc, const int* member_rank /*[n_sm], -1 = not a member*/,
                                 unsigned int n_members, uint8_t* buf, size_t n_chunks, const uint32_t* list,
                                 size_t n_work, int lines_per_chunk, int reps, uint32_t* cycles) {
    const int rank = member_rank[smid()];
    pin_rendezvous(pc, rank >= 0, n_members, 200000ull);
    if (rank < 0 || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    uint32_t sink = 0;
    for (size_t w = (size_t)rank; w < n_work; w += n_members) {
        const size_t c = list ? (size_t)list[w] : w;
        uint8_t* chunk = buf + c * AG_CHUNK_BYTES;
        uint8_t* partner = buf + (c ^ 1) * AG_CHUNK_BYTES;  // other chunk of the aligned pair: same large page
        if ((c ^ 1) >= n_chunks) partner = chunk + 3968;
        uint32_t best = 0xffffffffu;
        for (int l = 0; l < lines_per_chunk; ++l) {
            uint8_t* line = chunk + ((l * 1152 + 128) % AG_CHUNK_BYTES);
            for (int k = 0; k < reps; ++k) {
                const uint32_t saved = ld_cg_u32(line + lane * 4);
                __syncwarp();
                if (lane == 0) {
                    discard_l2_128(line);
                    sink += ld_cg_u32(partner);  // translation for this large page is now cached
                    best = min(best, timed_load_cg(line, sink));
                }
                __syncwarp();
                reinterpret_cast<uint32_t*>(line)[lane] = saved;
                __threadfence();
            }
        }
        if (lane == 0) cycles[w] = best;
    }
    if (lane == 0 && sink == 0x12345678u) cycles[0] = sink;
}

// ---- host helpers ------------------------------------------------------------------------------------
struct UnionFind {
    std::vector<int> p;
    explicit UnionFind(int n) : p(n) { std::iota(p.begin(), p.end(), 0); }
    int find(int x) { while (p[x] != x) { p[x] = p[p[x]]; x = p[x]; } return x; }
    void unite(int a, int b) { a = find(a); b = find(b); if (a != b) p[std::max(a, b)] = std::min(a, b); }
};

static void finish_counts(ag_topo_map* m) {
    memset(m->die_sm_count, 0, sizeof m->die_sm_count);
    memset(m->gpc_sm_count, 0, sizeof m->gpc_sm_count);
    m->n_unplaced = 0;
    for (int s = 0; s < m->n_sm; ++s) {
        m->die_sm_count[m->die[s] & 1]++;
        if (m->gpc[s] >= 0) m->gpc_sm_count[m->gpc[s]]++; else m->n_unplaced++;
    }
    for (int g = 0; g < m->n_gpc; ++g) {
        int c[2] = {0, 0};
        for (int s = 0; s < m->n_sm; ++s)
            if (m->gpc[s] == g) c[m->die[s] & 1]++;
        m->gpc_die[g] = c[1] > c[0] ? 1 : 0;
    }
}

}  // namespace ag

using namespace ag;

extern "C" ag_status ag_topo_from_observations(int32_t n_sm, const int32_t* cluster_sm, const int32_t* cluster_off,
                                               int32_t n_clusters, const uint32_t* lat, int32_t n_ref,
                                               ag_topo_map* map) {
    if (!map || n_sm <= 0 || n_sm > AG_MAX_SM || n_clusters < 0 || (n_clusters > 0 && (!cluster_sm || !cluster_off)))
        return AG_ERR_ARG;
    memset(map, 0, sizeof *map);
    map->n_sm = n_sm;
    map->n_tpc = (n_sm + 1) / 2;
    map->n_die = 2;
    for (int s = 0; s < n_sm; ++s) {
        map->tpc[s] = s / 2;  // two consecutive SM ids form a TPC (Section 5.1.2)
        map->gpc[s] = -1;
        map->is_random[s] = 1;
    }
    // GPC classes: SMs seen in one cluster share a GPC
    UnionFind uf(n_sm);
    std::vector<char> seen(n_sm, 0);
    for (int c = 0; c < n_clusters; ++c) {
        const int lo = cluster_off[c], hi = cluster_off[c + 1];
        if (hi - lo < 3) continue;  // pairs say nothing beyond the TPC
        for (int i = lo; i < hi; ++i) {
            const int s = cluster_sm[i];
            if (s < 0 || s >= n_sm) return AG_ERR_ARG;
            seen[s] = 1;
            uf.unite(cluster_sm[lo], s);
        }
    }
    int n_gpc = 0;
    std::vector<int> root_gpc(n_sm, -1);
    for (int s = 0; s < n_sm; ++s) {
        if (!seen[s]) continue;
        map->is_random[s] = 0;
        const int r = uf.find(s);
        if (root_gpc[r] < 0) {
            if (n_gpc >= AG_MAX_GPC) return AG_ERR_ARG;
            root_gpc[r] = n_gpc++;
        }
        map->gpc[s] = root_gpc[r];
    }
    map->n_gpc = n_gpc;
    if (n_clusters > 0) map->flags |= AG_TOPO_CLUSTER;
    // dies: SM s sits on SM 0's die when it sees every reference line at about the latency SM 0
    // sees it (within 25 %), and on the other die when it sees nearly every line very differently.
    // Comparing line by line keeps the split independent of whether a given line happened to be
    // served by L2 or by HBM: that depends on the line, not on the SM.
    if (lat && n_ref > 0) {
        int other = -1;
        for (int s = 0; s < n_sm; ++s) {
            int similar = 0;
            for (int r = 0; r < n_ref; ++r) {
                const double a = lat[(size_t)s * n_ref + r], b = lat[r];
                similar += (a <= 1.25 * b && b <= 1.25 * a);
            }
            if (similar * 4 > n_ref && similar * 4 < 3 * n_ref) {
                if (getenv("AG_DEBUG")) {
                    fprintf(stderr, "[ag] SM %d is like SM 0 on %d of %d lines; row:", s, similar, n_ref);
                    for (int r = 0; r < n_ref; ++r) fprintf(stderr, " %u", lat[(size_t)s * n_ref + r]);
                    fprintf(stderr, "\n[ag] SM 0 row:");
                    for (int r = 0; r < n_ref; ++r) fprintf(stderr, " %u", lat[r]);
                    fprintf(stderr, "\n");
                }
                return AG_ERR_NOISY_PROBE;
            }
            map->die[s] = similar * 2 >= n_ref ? 0 : 1;
            if (map->die[s] == 1 && other < 0) other = s;
        }
        if (other < 0) return AG_ERR_NOISY_PROBE;  // no second latency tier seen from any SM
        std::vector<uint32_t> nearv, farv;
        for (int r = 0; r < n_ref; ++r) {
            const uint32_t a = lat[r], b = lat[(size_t)other * n_ref + r];
            nearv.push_back(std::min(a, b));
            farv.push_back(std::max(a, b));
        }
        std::sort(nearv.begin(), nearv.end());
        std::sort(farv.begin(), farv.end());
        map->lat_near_cycles = nearv[n_ref / 2];
        map->lat_far_cycles = farv[n_ref / 2];
        map->lat_threshold = (map->lat_near_cycles + map->lat_far_cycles) / 2;
        map->flags |= AG_TOPO_LATENCY;
    }
    finish_counts(map);
    return AG_OK;
}

extern "C" int32_t ag_topo_place_by_gain(const double* gain, int32_t n, double solo_bw) {
    if (!gain || n <= 0 || solo_bw <= 0) return -1;
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (gain[i] < gain[best]) best = i;
    double runner = 1e300;
    for (int i = 0; i < n; ++i)
        if (i != best) runner = std::min(runner, gain[i]);
    // contended: the GPC's port to L2 was already full, so the TPC adds next to nothing; a TPC of
    // another GPC still adds a good part of its own bandwidth
    if (gain[best] < 0.35 * solo_bw && (n == 1 || runner > gain[best] + 0.20 * solo_bw)) return best;
    return -1;
}

namespace {

struct Scratch {
    PinCtrl* pc = nullptr;
    int* d_int = nullptr;
    uint8_t* ref = nullptr;
    long long* d_off = nullptr;
    uint32_t* d_out = nullptr;
    unsigned long long* d_mask = nullptr;
    uint4* bw_buf = nullptr;
    unsigned int* d_sink = nullptr;
    ~Scratch() {
        cudaFree(pc); cudaFree(d_int); cudaFree(ref); cudaFree(d_off); cudaFree(d_out); cudaFree(d_mask);
        cudaFree(bw_buf); cudaFree(d_sink);
    }
};

ag_status warm_up(int n_sm, float* d_sink) {
    k_warm_up<<<n_sm, 128>>>(30000000ull, d_sink);
    count_launch();
    AG_CUDA(cudaGetLastError());
    AG_CUDA(cudaDeviceSynchronize());
    return AG_OK;
}

ag_status set_pin_smem() {
    static std::atomic<unsigned long long> done{0};
    const cudaError_t e = once_per_device(done, [] {
        cudaError_t r = cudaFuncSetAttribute(k_census, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_cluster_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_latency_from_sm, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_l2_bandwidth, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_affinity_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_die_bandwidth, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem);
        return r;
    });
    return e == cudaSuccess ? AG_OK : cuda_fail(e);
}

// aggregate L2 read bandwidth (bytes/s) of the SMs in `mask`, best of `tries`
ag_status measure_bw(Scratch& sc, int n_sm, const unsigned long long mask[4], size_t slice_vec, int passes, int tries,
                     double* bw) {
    unsigned int n_members = 0;
    for (int s = 0; s < n_sm; ++s) n_members += (mask[s >> 6] >> (s & 63)) & 1ull;
    AG_CUDA(cudaMemcpy(sc.d_mask, mask, 4 * sizeof(unsigned long long), cudaMemcpyHostToDevice));
    double best = 0;
    std::vector<PinCtrl> h(1);
    for (int t = 0; t < tries; ++t) {
        AG_CUDA(cudaMemset(sc.pc, 0, sizeof(PinCtrl)));
        k_l2_bandwidth<<<n_sm, 1024, kPinSmem>>>(sc.pc, sc.d_mask, n_members, sc.bw_buf, slice_vec, passes, sc.d_sink);
        count_launch();
        AG_CUDA(cudaGetLastError());
        AG_CUDA(cudaDeviceSynchronize());
        AG_CUDA(cudaMemcpy(h.data(), sc.pc, sizeof(PinCtrl), cudaMemcpyDeviceToHost));
        unsigned long long t0 = ~0ull, t1 = 0;
        unsigned int got = 0;
        for (int s = 0; s < n_sm; ++s)
            if ((mask[s >> 6] >> (s & 63)) & 1ull) {
                if (h[0].t_end[s] == 0) continue;
                ++got;
                t0 = std::min(t0, h[0].t_start[s]);
                t1 = std::max(t1, h[0].t_end[s]);
            }
        if (got != n_members || t1 <= t0) continue;  // an SM of the set got no block: try again
        const double bytes = (double)n_members * passes * slice_vec * 16.0;
        best = std::max(best, bytes / ((double)(t1 - t0) * 1e-9));
    }
    *bw = best;
    return best > 0 ? AG_OK : AG_ERR_UNMANNED_SM;
}

ag_status latency_rows(Scratch& sc, int n_sm, const std::vector<int>& sms, int n_lines, int mode, int reps,
                       std::vector<uint32_t>& out /* sms.size() x n_lines */) {
    out.assign(sms.size() * (size_t)n_lines, 0);
    for (size_t i = 0; i < sms.size(); ++i) {
        bool ok = false;
        for (int attempt = 0; attempt < 3 && !ok; ++attempt) {
            AG_CUDA(cudaMemset(sc.pc, 0, sizeof(PinCtrl)));
            AG_CUDA(cudaMemset(sc.d_out, 0, sizeof(uint32_t) * n_lines));
            k_latency_from_sm<<<n_sm, 32, kPinSmem>>>(sc.pc, sms[i], sc.ref, sc.d_off, n_lines, reps, mode, sc.d_out, nullptr);
            count_launch();
            AG_CUDA(cudaGetLastError());
            AG_CUDA(cudaDeviceSynchronize());
            AG_CUDA(cudaMemcpy(&out[i * n_lines], sc.d_out, sizeof(uint32_t) * n_lines, cudaMemcpyDeviceToHost));
            ok = out[i * n_lines] != 0;  // zero: no block landed on that SM
        }
        if (!ok) return AG_ERR_UNMANNED_SM;
    }
    return AG_OK;
}

}  // namespace

extern "C" ag_status ag_topo_discover_phases(ag_topo_map* map, uint32_t phases) {
    if (!map) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    st = set_pin_smem();
    if (st != AG_OK) return st;
    int dev = 0, n_sm = 0, clock_khz = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    AG_CUDA(cudaDeviceGetAttribute(&clock_khz, cudaDevAttrClockRate, dev));
    if (n_sm > AG_MAX_SM) return AG_ERR_ARG;

    Scratch sc;
    const size_t ref_bytes = 8u << 20;
    AG_CUDA(cudaMalloc(&sc.pc, sizeof(PinCtrl)));
    AG_CUDA(cudaMalloc(&sc.d_int, sizeof(int) * 16384));
    AG_CUDA(cudaMalloc(&sc.ref, ref_bytes));
    AG_CUDA(cudaMemset(sc.ref, 0, ref_bytes));
    AG_CUDA(cudaMalloc(&sc.d_off, sizeof(long long) * 1024));
    AG_CUDA(cudaMalloc(&sc.d_out, sizeof(uint32_t) * 1024));
    AG_CUDA(cudaMalloc(&sc.d_mask, 4 * sizeof(unsigned long long)));
    AG_CUDA(cudaMalloc(&sc.d_sink, 64));

    st = warm_up(n_sm, reinterpret_cast<float*>(sc.d_sink));
    if (st != AG_OK) return st;
    // ---- census: every SM id exactly once
    AG_CUDA(cudaMemset(sc.pc, 0, sizeof(PinCtrl)));
    AG_CUDA(cudaMemset(sc.d_int, 0, sizeof(int) * AG_MAX_SM));
    k_census<<<n_sm, 32, kPinSmem>>>(sc.pc, sc.d_int, (unsigned int)n_sm);
    count_launch();
    AG_CUDA(cudaGetLastError());
    AG_CUDA(cudaDeviceSynchronize());
    std::vector<int> cnt(AG_MAX_SM);
    AG_CUDA(cudaMemcpy(cnt.data(), sc.d_int, sizeof(int) * AG_MAX_SM, cudaMemcpyDeviceToHost));
    for (int s = 0; s < AG_MAX_SM; ++s)
        if (cnt[s] != (s < n_sm ? 1 : 0)) return AG_ERR_UNMANNED_SM;

    // ---- cluster probing, sizes 3..8
    std::vector<int32_t> cl_sm, cl_off(1, 0);
    if (phases & AG_TOPO_CLUSTER) {
        for (int rep = 0; rep < 3; ++rep)
            for (int cs = 3; cs <= 8; ++cs) {
                const int n_clusters = std::max(1, (2 * n_sm) / cs);
                const int grid = n_clusters * cs;
                if (grid > 16384) continue;
                cudaLaunchConfig_t cfg;
                memset(&cfg, 0, sizeof cfg);
                cfg.gridDim = dim3(grid);
                cfg.blockDim = dim3(32);
                cfg.dynamicSmemBytes = kPinSmem;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = cs;
                attr[0].val.clusterDim.y = 1;
                attr[0].val.clusterDim.z = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
                AG_CUDA(cudaMemset(sc.d_int, 0xFF, sizeof(int) * grid));
                cudaError_t e = cudaLaunchKernelEx(&cfg, k_cluster_probe, sc.d_int);
                if (e != cudaSuccess) { cudaGetLastError(); continue; }  // this cluster size cannot be placed
                count_launch();
                AG_CUDA(cudaDeviceSynchronize());
                std::vector<int> ids(grid);
                AG_CUDA(cudaMemcpy(ids.data(), sc.d_int, sizeof(int) * grid, cudaMemcpyDeviceToHost));
                for (int c = 0; c < n_clusters; ++c) {
                    for (int i = 0; i < cs; ++i) cl_sm.push_back(ids[c * cs + i]);
                    cl_off.push_back((int32_t)cl_sm.size());
                }
            }
    }

    // ---- latency from every SM to the reference chunks
    std::vector<uint32_t> lat;
    std::vector<long long> offs(kRefChunks);
    if (phases & AG_TOPO_LATENCY) {
        const long long n_chunks = (long long)(ref_bytes / AG_CHUNK_BYTES);
        for (int r = 0; r < kRefChunks; ++r) offs[r] = ((r * 29LL + 3) % n_chunks) * AG_CHUNK_BYTES + 512;
        AG_CUDA(cudaMemcpy(sc.d_off, offs.data(), sizeof(long long) * kRefChunks, cudaMemcpyHostToDevice));
        std::vector<int> all(n_sm);
        std::iota(all.begin(), all.end(), 0);
        st = latency_rows(sc, n_sm, all, kRefChunks, 0, kLatReps, lat);
        if (st != AG_OK) return st;
    }
    st = ag_topo_from_observations(n_sm, cl_sm.data(), cl_off.data(), (int32_t)cl_off.size() - 1,
                                   lat.empty() ? nullptr : lat.data(), lat.empty() ? 0 : kRefChunks, map);
    if (st != AG_OK) return st;
    map->device = dev;
    map->sm_clock_khz = (uint32_t)clock_khz;
    map->flags |= AG_TOPO_CENSUS;

    // ---- L2-hit latency, same-die and other-die reader (appendix, L2 latency kernel)
    if ((phases & AG_TOPO_LATENCY) && map->die_sm_count[0] > 0 && map->die_sm_count[1] > 0) {
        int other = -1;
        for (int s = 0; s < n_sm && other < 0; ++s)
            if (map->die[s] == 1) other = s;
        // lines that are near for die 0
        std::vector<long long> near_off;
        if (other >= 0)
            for (int r = 0; r < kRefChunks; ++r)
                if (lat[r] < lat[(size_t)other * kRefChunks + r]) near_off.push_back(offs[r] + 1024);
        if (near_off.size() >= 4 && other >= 0) {
            const int n = (int)near_off.size();
            AG_CUDA(cudaMemcpy(sc.d_off, near_off.data(), sizeof(long long) * n, cudaMemcpyHostToDevice));
            std::vector<uint32_t> nearv, farv;
            // SM 0 rewrites each line (now dirty in its home L2 on die 0) and times a reload: local hit.
            st = latency_rows(sc, n_sm, std::vector<int>{0}, n, 2, 2, nearv);
            // An SM of the other die then loads each line once: it comes from the home partition
            // across the die-to-die fabric (a second load would hit the copy replicated locally).
            if (st == AG_OK) st = latency_rows(sc, n_sm, std::vector<int>{other}, n, 1, 1, farv);
            if (st != AG_OK) return st;
            std::sort(nearv.begin(), nearv.end());
            std::sort(farv.begin(), farv.end());
            // reported only when the two tiers are apart: lines that an earlier access already
            // replicated into the other die's L2 would read as local hits there
            if (farv[n / 2] > 1.3 * nearv[n / 2]) {
                map->l2_near_cycles = nearv[n / 2];
                map->l2_far_cycles = farv[n / 2];
            }
        }
    }

    // ---- place the random TPCs by L2-bandwidth contention (Section 5.1.2)
    // The known SMs of a GPC are run alone and together with the TPC.  Where the known SMs already
    // fill the GPC's port to L2, a TPC of the same GPC adds next to nothing while a TPC of another
    // GPC adds a good part of its own bandwidth.  GPCs whose known SMs do not fill the port cannot
    // be tested that way; a TPC that contends with no testable GPC of its die is placed by
    // elimination when exactly one such GPC with room for it (at most 10 TPCs per GPC) is left.
    if ((phases & AG_TOPO_BANDWIDTH) && (map->flags & AG_TOPO_CLUSTER) && (map->flags & AG_TOPO_LATENCY) &&
        map->n_unplaced > 0 && map->n_gpc > 0) {
        const size_t slice_bytes = 1u << 20;  // per-SM slice: larger than L1, 64 slices fit well inside L2
        const size_t slice_vec = slice_bytes / 16;
        AG_CUDA(cudaMalloc(&sc.bw_buf, slice_bytes * 64));
        AG_CUDA(cudaMemset(sc.bw_buf, 1, slice_bytes * 64));
        const int passes = 8, tries = 3;
        const bool dbg = getenv("AG_DEBUG") != nullptr;
        std::vector<double> base_bw(map->n_gpc, 0.0);
        std::vector<int> size_now(map->n_gpc, 0);
        auto mask_of_gpc = [&](int g, unsigned long long m[4]) {
            m[0] = m[1] = m[2] = m[3] = 0;
            for (int s = 0; s < n_sm; ++s)
                if (map->gpc[s] == g && !map->is_random[s]) m[s >> 6] |= 1ull << (s & 63);
        };
        double cap = 0;
        for (int g = 0; g < map->n_gpc; ++g) {
            unsigned long long mg[4];
            mask_of_gpc(g, mg);
            size_now[g] = map->gpc_sm_count[g];
            if (measure_bw(sc, n_sm, mg, slice_vec, passes, tries, &base_bw[g]) != AG_OK) base_bw[g] = 0;
            cap = std::max(cap, base_bw[g]);
        }
        for (int t = 0; t < map->n_tpc; ++t) {
            const int s0 = 2 * t, s1 = 2 * t + 1;
            if (s0 >= n_sm || map->gpc[s0] >= 0) continue;
            const int tpc_sms = s1 < n_sm ? 2 : 1;
            unsigned long long m[4] = {0, 0, 0, 0};
            m[s0 >> 6] |= 1ull << (s0 & 63);
            if (s1 < n_sm) m[s1 >> 6] |= 1ull << (s1 & 63);
            double solo = 0;
            if (measure_bw(sc, n_sm, m, slice_vec, passes, tries, &solo) != AG_OK) continue;
            std::vector<int> tested, untested;
            std::vector<double> gains;
            for (int g = 0; g < map->n_gpc; ++g) {
                if (map->gpc_die[g] != map->die[s0]) continue;   // a TPC sits on the die its latency shows
                if (size_now[g] + tpc_sms > 20) continue;        // a GPC holds at most 10 TPCs
                if (base_bw[g] < 0.93 * cap) { untested.push_back(g); continue; }  // port not full: no signal
                unsigned long long mg[4];
                mask_of_gpc(g, mg);
                for (int i = 0; i < 4; ++i) mg[i] |= m[i];
                double with = 0;
                if (measure_bw(sc, n_sm, mg, slice_vec, passes, tries, &with) != AG_OK) continue;
                tested.push_back(g);
                gains.push_back(with - base_bw[g]);
            }
            int pick_gpc = -1;
            const int pick = ag_topo_place_by_gain(gains.data(), (int)gains.size(), solo);
            if (pick >= 0) {
                pick_gpc = tested[pick];
            } else {
                bool any_low = false;
                for (double gn : gains) any_low |= gn < 0.35 * solo;
                if (!any_low && untested.size() == 1) pick_gpc = untested[0];
            }
            if (dbg) {
                fprintf(stderr, "[ag] TPC %d solo %.1f GB/s:", t, solo * 1e-9);
                for (size_t i = 0; i < tested.size(); ++i)
                    fprintf(stderr, " gpc%d base %.1f gain %.1f;", tested[i], base_bw[tested[i]] * 1e-9, gains[i] * 1e-9);
                for (int g : untested) fprintf(stderr, " gpc%d untested (base %.1f);", g, base_bw[g] * 1e-9);
                fprintf(stderr, " -> gpc %d\n", pick_gpc);
            }
            if (pick_gpc >= 0) {
                map->gpc[s0] = pick_gpc;
                if (s1 < n_sm) map->gpc[s1] = pick_gpc;
                size_now[pick_gpc] += tpc_sms;
            }
        }
        map->flags |= AG_TOPO_BANDWIDTH;
        finish_counts(map);
    }
    return AG_OK;
}

extern "C" ag_status ag_probe_latency_samples(int sm, int mode, int n_lines, int reps, uint32_t* cycles) {
    if (!cycles || n_lines < 1 || n_lines > 1024 || reps < 1 || reps > 64 || (mode < 0 || mode > 2)) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    st = set_pin_smem();
    if (st != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (sm < 0 || sm >= n_sm) return AG_ERR_ARG;
    Scratch sc;
    const size_t ref_bytes = 8u << 20;
    uint32_t* d_raw = nullptr;
    AG_CUDA(cudaMalloc(&sc.pc, sizeof(PinCtrl)));
    AG_CUDA(cudaMalloc(&sc.ref, ref_bytes));
    AG_CUDA(cudaMemset(sc.ref, 0, ref_bytes));
    AG_CUDA(cudaMalloc(&sc.d_off, sizeof(long long) * 1024));
    AG_CUDA(cudaMalloc(&sc.d_out, sizeof(uint32_t) * 1024 * 65));
    d_raw = sc.d_out + 1024;
    AG_CUDA(cudaMalloc(&sc.d_sink, 64));
    std::vector<long long> offs(n_lines);
    const long long n_chunks = (long long)(ref_bytes / AG_CHUNK_BYTES);
    for (int r = 0; r < n_lines; ++r) offs[r] = ((r * 29LL + 3) % n_chunks) * AG_CHUNK_BYTES + 512;
    AG_CUDA(cudaMemcpy(sc.d_off, offs.data(), sizeof(long long) * n_lines, cudaMemcpyHostToDevice));
    st = warm_up(n_sm, reinterpret_cast<float*>(sc.d_sink));
    if (st != AG_OK) return st;
    AG_CUDA(cudaMemset(sc.pc, 0, sizeof(PinCtrl)));
    AG_CUDA(cudaMemset(sc.d_out, 0, sizeof(uint32_t) * 1024 * 65));
    k_latency_from_sm<<<n_sm, 32, kPinSmem>>>(sc.pc, sm, sc.ref, sc.d_off, n_lines, reps, mode, sc.d_out, d_raw);
    count_launch();
    AG_CUDA(cudaGetLastError());
    AG_CUDA(cudaDeviceSynchronize());
    AG_CUDA(cudaMemcpy(cycles, d_raw, sizeof(uint32_t) * n_lines * reps, cudaMemcpyDeviceToHost));
    return cycles[0] ? AG_OK : AG_ERR_UNMANNED_SM;
}

extern "C" ag_status ag_probe_l2_bandwidth(const uint64_t sm_mask[4], double* bytes_per_s) {
    if (!sm_mask || !bytes_per_s) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    st = set_pin_smem();
    if (st != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    unsigned long long m[4] = {sm_mask[0], sm_mask[1], sm_mask[2], sm_mask[3]};
    unsigned int members = 0;
    for (int s = 0; s < AG_MAX_SM; ++s) {
        const bool in = (m[s >> 6] >> (s & 63)) & 1ull;
        if (in && s >= n_sm) return AG_ERR_ARG;
        members += in;
    }
    if (members == 0) return AG_ERR_ARG;
    Scratch sc;
    const size_t slice_bytes = 1u << 20;
    AG_CUDA(cudaMalloc(&sc.pc, sizeof(PinCtrl)));
    AG_CUDA(cudaMalloc(&sc.d_mask, 4 * sizeof(unsigned long long)));
    AG_CUDA(cudaMalloc(&sc.d_sink, 64));
    AG_CUDA(cudaMalloc(&sc.bw_buf, slice_bytes * 64));
    AG_CUDA(cudaMemset(sc.bw_buf, 1, slice_bytes * 64));
    return measure_bw(sc, n_sm, m, slice_bytes / 16, 8, 3, bytes_per_s);
}

extern "C" ag_status topo_discover(ag_topo_map* map) {
    return ag_topo_discover_phases(map, AG_TOPO_CENSUS | AG_TOPO_CLUSTER | AG_TOPO_LATENCY | AG_TOPO_BANDWIDTH);
}

// ---- affinity --------------------------------------------------------------------------------------------
// Probes all chunks (list == nullptr) or the listed ones from the SMs of one die; cycles gets one entry per
// probed chunk (in list order when a list is given).
static ag_status probe_from_die(uint8_t* buf, size_t n_chunks, const ag_topo_map* map, int die,
                                std::vector<uint32_t>& cycles, int ref_sm[2],
                                const std::vector<uint32_t>* list = nullptr, int lines = 2, int reps = 3) {
    ag_status st = set_pin_smem();
    if (st != AG_OK) return st;
    const int n_sm = map->n_sm;
    std::vector<int> rank(AG_MAX_SM, -1);
    unsigned int n_members = 0;
    for (int s = 0; s < n_sm; ++s)
        if (map->die[s] == die) {
            if (ref_sm[die] < 0) ref_sm[die] = s;
            rank[s] = (int)n_members++;
        }
    if (n_members == 0) return AG_ERR_ARG;
    PinCtrl* pc = nullptr;
    int* d_rank = nullptr;
    uint32_t* d_cycles = nullptr;
    uint32_t* d_list = nullptr;
    const size_t n_work = list ? list->size() : n_chunks;
    if (n_work < n_members) n_members = (unsigned int)std::max<size_t>(1, n_work);  // fewer chunks than SMs: fewer workers
    for (int s = 0; s < n_sm; ++s)
        if (rank[s] >= (int)n_members) rank[s] = -1;
    cudaError_t e = cudaSuccess;
    do {
        if ((e = cudaMalloc(&pc, sizeof(PinCtrl))) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_rank, sizeof(int) * AG_MAX_SM)) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_cycles, sizeof(uint32_t) * n_work)) != cudaSuccess) break;
        if (list) {
            if ((e = cudaMalloc(&d_list, sizeof(uint32_t) * n_work)) != cudaSuccess) break;
            if ((e = cudaMemcpy(d_list, list->data(), sizeof(uint32_t) * n_work, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        }
        if ((e = cudaMemset(pc, 0, sizeof(PinCtrl))) != cudaSuccess) break;
        if ((e = cudaMemset(d_cycles, 0, sizeof(uint32_t) * n_work)) != cudaSuccess) break;
        if ((e = cudaMemcpy(d_rank, rank.data(), sizeof(int) * AG_MAX_SM, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        k_affinity_probe<<<n_sm, 32, kPinSmem>>>(pc, d_rank, n_members, buf, n_chunks, d_list, n_work, lines, reps, d_cycles);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) break;
        if ((e = cudaDeviceSynchronize()) != cudaSuccess) break;
        cycles.resize(n_work);
        e = cudaMemcpy(cycles.data(), d_cycles, sizeof(uint32_t) * n_work, cudaMemcpyDeviceToHost);
    } while (0);
    cudaFree(pc);
    cudaFree(d_rank);
    cudaFree(d_cycles);
    cudaFree(d_list);
    if (e != cudaSuccess) return cuda_fail(e);
    for (uint32_t c : cycles)
        if (c == 0) return AG_ERR_UNMANNED_SM;  // a member SM got no block: its chunks were not probed
    return AG_OK;
}

// A chunk belongs to the die whose SMs reach it faster (Section 6.1.1; the appendix on multi-tier
// parts assigns each address to the group with the lowest latency in the same way).
static ag_status classify(const std::vector<uint32_t>& c0, const std::vector<uint32_t>& c1,
                          std::vector<uint8_t>& table, size_t* ambiguous) {
    table.resize(c0.size());
    size_t amb = 0;
    for (size_t i = 0; i < c0.size(); ++i) {
        table[i] = c0[i] <= c1[i] ? 0 : 1;
        const double lo = std::min(c0[i], c1[i]), hi = std::max(c0[i], c1[i]);
        if (hi < 1.25 * lo) ++amb;
    }
    *ambiguous = amb;
    return amb * 50 > c0.size() ? AG_ERR_NOISY_PROBE : AG_OK;  // more than 2 % undecided
}

extern "C" ag_status ag_affinity_from_table(const void* buf, size_t bytes, const uint8_t* die_of_chunk,
                                            size_t n_chunks, ag_affinity_map** out) {
    if (!out || !die_of_chunk || n_chunks == 0 || bytes != n_chunks * AG_CHUNK_BYTES) return AG_ERR_ARG;
    *out = nullptr;
    ag_affinity_map* a = new (std::nothrow) ag_affinity_map();
    if (!a) return AG_ERR_NOMEM;
    a->base = buf;
    a->bytes = bytes;
    a->n_chunks = n_chunks;
    a->d_die_of_chunk = nullptr;
    a->h_die_of_chunk.assign(die_of_chunk, die_of_chunk + n_chunks);
    for (auto& v : a->h_die_of_chunk) v = v ? 1 : 0;
    a->ref_sm[0] = a->ref_sm[1] = -1;
    a->n_ambiguous = 0;
    cudaError_t e = cudaMalloc(&a->d_die_of_chunk, n_chunks);
    if (e == cudaSuccess) e = cudaMemcpy(a->d_die_of_chunk, a->h_die_of_chunk.data(), n_chunks, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        ag_affinity_destroy(a);
        return cuda_fail(e);
    }
    *out = a;
    return AG_OK;
}

extern "C" ag_status ag_affinity_probe_with_map(void* buf, size_t bytes, const ag_topo_map* map,
                                                ag_affinity_map** out) {
    if (!buf || !map || !out || bytes == 0 || (bytes % AG_CHUNK_BYTES) || ((uintptr_t)buf % AG_CHUNK_BYTES))
        return AG_ERR_ARG;
    *out = nullptr;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    if (!(map->flags & AG_TOPO_LATENCY)) return AG_ERR_ARG;
    const size_t n_chunks = bytes / AG_CHUNK_BYTES;
    std::vector<uint32_t> cycles;
    int ref_sm[2] = {-1, -1};
    {
        float* d_sink = nullptr;
        AG_CUDA(cudaMalloc(&d_sink, 64));
        st = warm_up(map->n_sm, d_sink);
        cudaFree(d_sink);
        if (st != AG_OK) return st;
    }
    std::vector<uint32_t> cycles1;
    st = probe_from_die((uint8_t*)buf, n_chunks, map, 0, cycles, ref_sm);
    if (st != AG_OK) return st;
    st = probe_from_die((uint8_t*)buf, n_chunks, map, 1, cycles1, ref_sm);
    if (st != AG_OK) return st;
    // chunks whose two latencies are less than 25 % apart are probed once more, with more lines and repeats;
    // the smaller of the old and the new value is kept for each die
    {
        std::vector<uint32_t> again;
        for (size_t i = 0; i < n_chunks; ++i) {
            const double lo = std::min(cycles[i], cycles1[i]), hi = std::max(cycles[i], cycles1[i]);
            if (hi < 1.25 * lo) again.push_back((uint32_t)i);
        }
        if (!again.empty() && again.size() * 20 < n_chunks) {
            std::vector<uint32_t> r0, r1;
            int dummy[2] = {0, 0};
            st = probe_from_die((uint8_t*)buf, n_chunks, map, 0, r0, dummy, &again, 6, 4);
            if (st == AG_OK) st = probe_from_die((uint8_t*)buf, n_chunks, map, 1, r1, dummy, &again, 6, 4);
            if (st != AG_OK) return st;
            for (size_t k = 0; k < again.size(); ++k) {
                cycles[again[k]] = std::min(cycles[again[k]], r0[k]);
                cycles1[again[k]] = std::min(cycles1[again[k]], r1[k]);
            }
        }
    }
    std::vector<uint8_t> table;
    size_t ambiguous = 0;
    st = classify(cycles, cycles1, table, &ambiguous);
    if (st != AG_OK) return st;
    st = ag_affinity_from_table(buf, bytes, table.data(), n_chunks, out);
    if (st != AG_OK) return st;
    (*out)->h_cycles.swap(cycles);
    (*out)->h_cycles1.swap(cycles1);
    (*out)->ref_sm[0] = ref_sm[0];
    (*out)->ref_sm[1] = ref_sm[1];
    (*out)->n_ambiguous = ambiguous;
    return AG_OK;
}

extern "C" ag_status affinity_probe(void* buf, size_t bytes, ag_affinity_map** out) {
    ag_topo_map map;
    ag_status st = ag_topo_discover_phases(&map, AG_TOPO_CENSUS | AG_TOPO_LATENCY);
    if (st != AG_OK) return st;
    return ag_affinity_probe_with_map(buf, bytes, &map, out);
}

extern "C" ag_status ag_affinity_check_complement(const ag_affinity_map* amap, const ag_topo_map* map,
                                                  size_t* mismatches) {
    (void)map;
    if (!amap || !mismatches || amap->h_cycles.empty()) return AG_ERR_ARG;
    *mismatches = amap->n_ambiguous;
    return AG_OK;
}

// Section 6.1.2: the partition is the parity of a subset of address bits.  Inside one 2 MiB page (512 chunks,
// physically contiguous) the die of chunk i is parity(i & mask) ^ c with a page-independent mask over the nine
// chunk-index bits (address bits 12..20) and a per-page constant c that absorbs the higher address bits.
extern "C" ag_status ag_affinity_fit_hash(const ag_affinity_map* amap, uint32_t* mask_out, size_t* violations) {
    if (!amap || !mask_out) return AG_ERR_ARG;
    const size_t per_page = (2u << 20) / AG_CHUNK_BYTES;  // 512
    // chunk index inside its 2 MiB page follows from the address, not from the position in the buffer
    const size_t first = ((uintptr_t)amap->base / AG_CHUNK_BYTES) % per_page;
    const std::vector<uint8_t>& die = amap->h_die_of_chunk;
    const size_t n = die.size();
    if (n < 2 * per_page) return AG_ERR_ARG;  // needs at least one complete page
    uint32_t mask = 0;
    for (int b = 0; b < 9; ++b) {
        size_t flips = 0, total = 0;
        for (size_t i = 0; i < n; ++i) {
            const size_t in_page = (first + i) % per_page;
            const size_t partner_in_page = in_page ^ (1u << b);
            const long long j = (long long)i + (long long)partner_in_page - (long long)in_page;
            if (j < 0 || (size_t)j >= n) continue;
            ++total;
            flips += die[i] != die[(size_t)j];
        }
        if (total && flips * 2 > total) mask |= 1u << b;  // flipping this bit changes the die: it is in the hash
    }
    *mask_out = mask;
    if (violations) {
        // per-page constant by majority, then count the chunks the fitted hash gets wrong
        size_t bad = 0;
        size_t i = 0;
        while (i < n) {
            const size_t in_page0 = (first + i) % per_page;
            const size_t len = std::min(n - i, per_page - in_page0);
            size_t ones = 0;
            for (size_t k = 0; k < len; ++k) ones += die[i + k] ^ (__builtin_popcount((uint32_t)(in_page0 + k) & mask) & 1);
            const uint8_t c = ones * 2 > len ? 1 : 0;
            for (size_t k = 0; k < len; ++k)
                bad += (die[i + k] ^ (__builtin_popcount((uint32_t)(in_page0 + k) & mask) & 1)) != c;
            i += len;
        }
        *violations = bad;
    }
    return AG_OK;
}

extern "C" ag_status ag_probe_cluster_layout(int cluster_size, int n_clusters, int32_t* cluster_of_sm) {
    if (!cluster_of_sm || cluster_size < 2 || cluster_size > 8 || n_clusters < 1 || n_clusters * cluster_size > 4096) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    static std::atomic<unsigned long long> attr_done{0};
    AG_CUDA(once_per_device(attr_done, [] { return cudaFuncSetAttribute(k_cluster_layout, cudaFuncAttributeMaxDynamicSharedMemorySize, kPinSmem); }));
    const int grid = n_clusters * cluster_size;
    int* d_smid = nullptr;
    unsigned long long* d_start = nullptr;
    unsigned int* d_started = nullptr;
    cudaError_t e = cudaMalloc(&d_smid, sizeof(int) * grid);
    if (e == cudaSuccess) e = cudaMalloc(&d_start, sizeof(unsigned long long) * grid);
    if (e == cudaSuccess) e = cudaMalloc(&d_started, sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(d_smid, 0xFF, sizeof(int) * grid);
    if (e == cudaSuccess) e = cudaMemset(d_started, 0, sizeof(unsigned int));
    std::vector<int> ids(grid, -1);
    std::vector<unsigned long long> t(grid, 0);
    if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(32);
        cfg.dynamicSmemBytes = kPinSmem;      // more than half an SM: one block per SM at a time
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = cluster_size;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, k_cluster_layout, d_smid, d_start, d_started, (unsigned int)grid);
        if (e == cudaSuccess) count_launch();
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(ids.data(), d_smid, sizeof(int) * grid, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(t.data(), d_start, sizeof(unsigned long long) * grid, cudaMemcpyDeviceToHost);
    cudaFree(d_smid);
    cudaFree(d_start);
    cudaFree(d_started);
    if (e != cudaSuccess) return cuda_fail(e);
    std::vector<unsigned long long> first(AG_MAX_SM, ~0ull);
    for (int s = 0; s < AG_MAX_SM; ++s) cluster_of_sm[s] = -1;
    for (int b = 0; b < grid; ++b) {
        const int s = ids[b];
        if (s < 0 || s >= AG_MAX_SM) continue;
        if (t[b] < first[s]) {                 // an SM may host a second cluster after the first has left: keep the first
            first[s] = t[b];
            cluster_of_sm[s] = b / cluster_size;
        }
    }
    return AG_OK;
}

extern "C" ag_status ag_probe_die_bandwidth(const ag_affinity_map* amap, const ag_topo_map* map, int reader_die,
                                            int chunk_die, double* bytes_per_s) {
    if (!amap || !map || !bytes_per_s || (reader_die | 1) != 1 || (chunk_die | 1) != 1 || !amap->base) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    st = set_pin_smem();
    if (st != AG_OK) return st;
    std::vector<uint32_t> list;
    for (size_t c = 0; c < amap->n_chunks; ++c)
        if (amap->h_die_of_chunk[c] == chunk_die) list.push_back((uint32_t)c);
    if (list.empty()) return AG_ERR_ARG;
    const int n_sm = map->n_sm;
    std::vector<int> rank(AG_MAX_SM, -1);
    unsigned int n_members = 0;
    for (int s = 0; s < n_sm; ++s)
        if (map->die[s] == reader_die) rank[s] = (int)n_members++;
    if (n_members == 0) return AG_ERR_ARG;
    PinCtrl* pc = nullptr;
    int* d_rank = nullptr;
    uint32_t* d_list = nullptr;
    unsigned int* d_sink = nullptr;
    cudaError_t e = cudaSuccess;
    double best = 0;
    do {
        if ((e = cudaMalloc(&pc, sizeof(PinCtrl))) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_rank, sizeof(int) * AG_MAX_SM)) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_list, sizeof(uint32_t) * list.size())) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_sink, 64)) != cudaSuccess) break;
        if ((e = cudaMemcpy(d_rank, rank.data(), sizeof(int) * AG_MAX_SM, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(d_list, list.data(), sizeof(uint32_t) * list.size(), cudaMemcpyHostToDevice)) != cudaSuccess) break;
        // enough passes to stream at least 1 GiB, so that the buffer cannot be served from L2 alone unless it is small
        const size_t bytes_per_pass = list.size() * (size_t)AG_CHUNK_BYTES;
        const int passes = (int)std::max<size_t>(1, (1ull << 30) / bytes_per_pass);
        std::vector<PinCtrl> h(1);
        for (int t = 0; t < 3 && e == cudaSuccess; ++t) {
            if ((e = cudaMemset(pc, 0, sizeof(PinCtrl))) != cudaSuccess) break;
            k_die_bandwidth<<<n_sm, 256, kPinSmem>>>(pc, d_rank, n_members, (const uint8_t*)amap->base, d_list, list.size(),
                                                    passes, d_sink);
            count_launch();
            if ((e = cudaGetLastError()) != cudaSuccess) break;
            if ((e = cudaDeviceSynchronize()) != cudaSuccess) break;
            if ((e = cudaMemcpy(h.data(), pc, sizeof(PinCtrl), cudaMemcpyDeviceToHost)) != cudaSuccess) break;
            unsigned long long t0 = ~0ull, t1 = 0;
            unsigned int got = 0;
            for (int s2 = 0; s2 < n_sm; ++s2)
                if (rank[s2] >= 0 && h[0].t_end[s2]) {
                    ++got;
                    t0 = std::min(t0, h[0].t_start[s2]);
                    t1 = std::max(t1, h[0].t_end[s2]);
                }
            if (got == n_members && t1 > t0)
                best = std::max(best, (double)bytes_per_pass * passes / ((double)(t1 - t0) * 1e-9));
        }
    } while (0);
    cudaFree(pc);
    cudaFree(d_rank);
    cudaFree(d_list);
    cudaFree(d_sink);
    if (e != cudaSuccess) return cuda_fail(e);
    *bytes_per_s = best;
    return best > 0 ? AG_OK : AG_ERR_UNMANNED_SM;
}

// ---- copy-ring bandwidth (the streaming kernels' ring without their arithmetic) --------------------------------
// Block b streams its own contiguous share of the buffer through a ring of `stages` shared-memory buffers of
// `stage_bytes`: warp w < producers refills the stages w, w + producers, ... with one bulk copy each, one thread of
// another warp takes them off in order, spends `hold_ns` on each (one after the other, like a thread that issues a
// stage's MMAs) and hands it back.  Every wait is bounded; a wait that runs out sets *err.
constexpr int kRingMaxStages = 8;
__global__ void __launch_bounds__(160, 1) k_ring_bandwidth(const uint8_t* __restrict__ src, long long n_stages, int stages, int stage_bytes,
                                                            int producers, int hold_ns, unsigned long long* t_out, int* err,
                                                            unsigned int* sink) {
    extern __shared__ __align__(1024) uint8_t ring_smem[];
    __shared__ uint64_t full[kRingMaxStages], empty[kRingMaxStages];
    const uint32_t raw = smem_u32(ring_smem);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(smem_u32(&full[i]), 1);
            mbar_init(smem_u32(&empty[i]), 1);
        }
        mbar_fence_init();
    }
    __syncthreads();
    volatile int* abort_flag = err;
    const uint64_t limit = 2000000000ull;
    const uint64_t stream_policy = l2_policy_evict_first();
    const uint8_t* mine = src + (size_t)blockIdx.x * (size_t)n_stages * (size_t)stage_bytes;
    const unsigned long long t0 = globaltimer_ns();
    if (warp < producers) {
        if (lane == 0) {
            for (long long c = warp; c < n_stages; c += producers) {
                const int st = (int)(c % stages);
                if (!mbar_wait(smem_u32(&empty[st]), (uint32_t)(((c / stages) & 1) ^ 1), abort_flag, limit)) break;
                mbar_expect_tx(smem_u32(&full[st]), (uint32_t)stage_bytes);
                bulk_load_hint(base + st * stage_bytes, mine + (size_t)c * stage_bytes, (uint32_t)stage_bytes, smem_u32(&full[st]), stream_policy);
            }
        }
    } else if (warp == producers) {
        if (lane == 0) {
            unsigned int acc = 0;
            for (long long c = 0; c < n_stages; ++c) {
                const int st = (int)(c % stages);
                if (!mbar_wait(smem_u32(&full[st]), (uint32_t)((c / stages) & 1), abort_flag, limit)) break;
                acc += *reinterpret_cast<volatile unsigned int*>(ring_smem + (base - raw) + st * stage_bytes + 64);
                if (hold_ns > 0) {
                    const unsigned long long h0 = globaltimer_ns();
                    while (globaltimer_ns() - h0 < (unsigned long long)hold_ns) {}
                }
                mbar_arrive(smem_u32(&empty[st]));
            }
            if (acc == 0x12345u) sink[0] = acc;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        t_out[2 * blockIdx.x] = t0;
        t_out[2 * blockIdx.x + 1] = globaltimer_ns();
    }
}

extern "C" ag_status ag_probe_ring_bandwidth(const void* buf, size_t bytes, int n_blocks, int stages, int stage_bytes, int producers,
                                             int hold_ns, double* bytes_per_s) {
    // producers <= stages: the one consuming thread hands the stages back in order, so a copying warp is never more than
    // one use of a stage ahead of that stage's barrier
    if (!buf || !bytes_per_s || ((uintptr_t)buf & 15u) || n_blocks < 1 || n_blocks > AG_MAX_SM || stages < 1 || stages > kRingMaxStages ||
        stage_bytes < 4096 || stage_bytes > 65536 || (stage_bytes & 4095) || stages * stage_bytes > 192 * 1024 || producers < 1 ||
        producers > 3 || producers > stages || hold_ns < 0 || hold_ns > 100000)
        return AG_ERR_ARG;
    const long long n_stages = (long long)(bytes / (size_t)n_blocks / (size_t)stage_bytes);
    if (n_stages < 1) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    static std::atomic<unsigned long long> attr_done{0};
    AG_CUDA(once_per_device(attr_done, [] { return cudaFuncSetAttribute(k_ring_bandwidth, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024); }));
    unsigned long long* d_t = nullptr;
    int* d_err = nullptr;
    unsigned int* d_sink = nullptr;
    cudaError_t e = cudaSuccess;
    double best = 0;
    int h_err = 0;
    do {
        if ((e = cudaMalloc(&d_t, sizeof(unsigned long long) * 2 * n_blocks)) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_err, sizeof(int))) != cudaSuccess) break;
        if ((e = cudaMalloc(&d_sink, 64)) != cudaSuccess) break;
        if ((e = cudaMemset(d_err, 0, sizeof(int))) != cudaSuccess) break;
        std::vector<unsigned long long> h(2 * (size_t)n_blocks);
        for (int t = 0; t < 3 && e == cudaSuccess && !h_err; ++t) {
            // 200 KB of shared memory per block: one block per SM
            k_ring_bandwidth<<<n_blocks, (producers + 1) * 32, 200 * 1024>>>((const uint8_t*)buf, n_stages, stages, stage_bytes, producers, hold_ns,
                                                                            d_t, d_err, d_sink);
            count_launch();
            if ((e = cudaGetLastError()) != cudaSuccess) break;
            if ((e = cudaDeviceSynchronize()) != cudaSuccess) break;
            if ((e = cudaMemcpy(h.data(), d_t, sizeof(unsigned long long) * h.size(), cudaMemcpyDeviceToHost)) != cudaSuccess) break;
            if ((e = cudaMemcpy(&h_err, d_err, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) break;
            unsigned long long t0 = ~0ull, t1 = 0;
            for (int b = 0; b < n_blocks; ++b) {
                t0 = std::min(t0, h[2 * b]);
                t1 = std::max(t1, h[2 * b + 1]);
            }
            if (t1 > t0) best = std::max(best, (double)n_stages * stage_bytes * n_blocks / ((double)(t1 - t0) * 1e-9));
        }
    } while (0);
    cudaFree(d_t);
    cudaFree(d_err);
    cudaFree(d_sink);
    if (e != cudaSuccess) return cuda_fail(e);
    if (h_err) return AG_ERR_TIMEOUT;
    *bytes_per_s = best;
    return AG_OK;
}

extern "C" ag_status ag_affinity_export(const ag_affinity_map* amap, uint8_t* die_of_chunk, size_t cap,
                                        size_t* n_chunks) {
    if (!amap) return AG_ERR_ARG;
    if (n_chunks) *n_chunks = amap->n_chunks;
    if (!die_of_chunk) return n_chunks ? AG_OK : AG_ERR_ARG;
    if (cap < amap->n_chunks) return AG_ERR_ARG;
    memcpy(die_of_chunk, amap->h_die_of_chunk.data(), amap->n_chunks);
    return AG_OK;
}

extern "C" ag_status ag_affinity_cycles(const ag_affinity_map* amap, uint32_t* cycles, size_t cap) {
    if (!amap || !cycles || amap->h_cycles.empty() || cap < 2 * amap->n_chunks) return AG_ERR_ARG;
    memcpy(cycles, amap->h_cycles.data(), amap->n_chunks * sizeof(uint32_t));
    memcpy(cycles + amap->n_chunks, amap->h_cycles1.data(), amap->n_chunks * sizeof(uint32_t));
    return AG_OK;
}

extern "C" void ag_affinity_destroy(ag_affinity_map* amap) {
    if (!amap) return;
    cudaFree(amap->d_die_of_chunk);
    delete amap;
}
