// Device-side pieces shared by the persistent kernels: joining the plan (which SM am I, is it
// planned, take its slot), and the source of work units (static per-SM list with adoption of
// unmanned lists, or dynamic pulls from the per-die queues).  Section 7.1.2 of the paper: one
// persistent block per SM that asks which SM it runs on and processes the tasks planned for it.
#pragma once
#include "internal.h"
#include "ptx.cuh"

namespace ag {

constexpr int kThreads = 192;       // warp 0 scheduler+producer, warp 1 MMA issuer, warps 2-5 epilogue
constexpr int kRing = 8;            // depth of the unit-id ring between the scheduler and its consumers
constexpr int kEpiWarps = 4;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every device-side wait gives up after 2 s

struct PersistParams {
    const int32_t* image;   // plan image (device)
    PlanCtrl* ctrl;
    int32_t* tile_owner;
    int32_t* tile_count;
    unsigned long long* unit_times;   // [n_units][2] start / end in ns of the global timer, or null (tracing off)
    int M, N, K;
    int b, n_units, n_sm;
    int tiles_n, k_splits, kslabs_total, kslabs_per_split;
    int static_assign;
    unsigned int epoch;
    unsigned long long wait_limit_ns;
    int b_blocks;           // 1: tm_b is the 3-D [N/64][K][64] view of B (one copy per k-slab)
};

__device__ __forceinline__ void report_timeout(const PersistParams& p, int role) {
    if (atomicCAS(&p.ctrl->status, 0, (int)AG_ERR_TIMEOUT) == 0) p.ctrl->status_info = (role << 16) | (int)smid();
}

// Dynamic mode: take the next index of a die's queue; the 64-bit head carries the epoch of the
// launch that last touched it, so it resets itself.  Returns -1 when the queue is drained.
__device__ inline int pop_queue(unsigned long long* head, unsigned int epoch, int len) {
    for (int tries = 0; tries < 100000; ++tries) {
        unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(head);
        if ((unsigned int)(cur >> 32) != epoch) {
            if (len <= 0) return -1;
            const unsigned long long nv = ((unsigned long long)epoch << 32) | 1ull;
            if (atomicCAS(head, cur, nv) == cur) return 0;
            continue;
        }
        const int idx = (int)(cur & 0xffffffffull);
        if (idx >= len) return -1;
        if (atomicCAS(head, cur, cur + 1) == cur) return idx;
    }
    return -1;
}

// Called by every thread of the block.  Returns the plan slot of this block's SM, or -1 if the
// block has nothing to do (SM not in the plan, or its slot already taken by another block).
// A block on an unplanned SM stays resident until every planned SM has a block (at most ~40 us),
// so that blocks still being placed can only land on SMs that have none yet.
__device__ inline int join_plan(const PersistParams& p, int* s_member) {
    const PlanLayout lay{p.b, p.n_units, p.n_sm};
    const int slot = p.image[lay.smid_to_slot() + (int)smid()];
    if (slot < 0) {
        const uint64_t t0 = globaltimer_ns();
        while (true) {
            int ok = 1;
            for (int i = threadIdx.x; i < p.b; i += blockDim.x)
                ok &= (*reinterpret_cast<volatile unsigned int*>(&p.ctrl->claimed[i]) == p.epoch);
            if (__syncthreads_and(ok)) break;
            if (globaltimer_ns() - t0 > 40000ull) break;
            __nanosleep(200);
        }
        return -1;
    }
    if (threadIdx.x == 0) *s_member = atomicMax(&p.ctrl->claimed[slot], p.epoch) < p.epoch;
    __syncthreads();
    return *s_member ? slot : -1;
}

// Source of work units for one block.  Warp-collective: every lane of the scheduler warp holds the
// same state and calls next() together; atomics are done by lane 0 and broadcast.
struct UnitSource {
    const PersistParams& p;
    PlanLayout lay;
    int idx, list_off, list_len, scan, dyn_die;

    __device__ UnitSource(const PersistParams& pp, int slot) : p(pp), lay{pp.b, pp.n_units, pp.n_sm} {
        idx = 0;
        list_off = p.image[lay.sm_q_off() + slot];
        list_len = p.image[lay.sm_q_off() + slot + 1] - list_off;
        scan = 0;
        dyn_die = p.image[lay.sm_die() + slot];
    }
    // next unit id, or -1 when there is nothing left for this block
    __device__ int next(int lane) {
        if (p.static_assign) {
            while (true) {
                if (idx < list_len) return p.image[lay.sm_q() + list_off + idx++];
                // Own list done: look for a planned SM that never got a block and run its list.  The 32
                // lanes check 32 claim flags at a time (a serial scan would cost one L2 round trip each).
                int cand = -1;
                for (; scan < p.b; scan += 32) {
                    const int i = scan + lane;
                    const bool unclaimed =
                        i < p.b && *reinterpret_cast<volatile unsigned int*>(&p.ctrl->claimed[i]) != p.epoch;
                    const unsigned m = __ballot_sync(0xffffffffu, unclaimed);
                    if (m) { cand = scan + __ffs(m) - 1; break; }
                }
                if (cand < 0) return -1;
                int got = 0;
                if (lane == 0) got = atomicMax(&p.ctrl->claimed[cand], p.epoch) < p.epoch;
                got = __shfl_sync(0xffffffffu, got, 0);
                if (got) {
                    list_off = p.image[lay.sm_q_off() + cand];
                    list_len = p.image[lay.sm_q_off() + cand + 1] - list_off;
                    idx = 0;
                    if (lane == 0) atomicAdd(&p.ctrl->adopted, 1u);
                }
            }
        }
        int u = -1;
        if (lane == 0) {
            for (int t = 0; t < 2 && u < 0; ++t) {
                const int q_off = p.image[lay.die_q_off() + dyn_die];
                const int q_len = p.image[lay.die_q_off() + dyn_die + 1] - q_off;
                const int e = pop_queue(&p.ctrl->die_head[dyn_die], p.epoch, q_len);
                if (e >= 0) u = p.image[lay.die_q() + q_off + e];
                else dyn_die ^= 1;  // own die drained: help the other one
            }
        }
        return __shfl_sync(0xffffffffu, u, 0);
    }
};

// Fills the launch parameters every persistent kernel needs from a plan (host).
inline PersistParams make_persist_params(const ag_plan* plan, int M, int N, int K) {
    PersistParams gp;
    gp.image = plan->d_image;
    gp.ctrl = plan->d_ctrl;
    gp.tile_owner = plan->d_tile_owner;
    gp.tile_count = plan->d_tile_count;
    gp.unit_times = plan->d_unit_times;
    gp.M = M; gp.N = N; gp.K = K;
    gp.b = plan->lay.b; gp.n_units = plan->lay.n_units; gp.n_sm = plan->lay.n_sm;
    gp.tiles_n = plan->header[H_TILES_N]; gp.k_splits = plan->header[H_KSPLITS];
    gp.kslabs_total = plan->kslabs_total; gp.kslabs_per_split = plan->kslabs_per_split;
    gp.static_assign = plan->header[H_STATIC];
    gp.epoch = ++plan->epoch;
    gp.wait_limit_ns = kWaitLimitNs;
    gp.b_blocks = 0;
    return gp;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_tiled();
// 2-D row-major tensor of `rows` x `cols` elements, box = box_cols x box_rows, 128-byte swizzle.
bool encode_2d(CUtensorMap* tm, CUtensorMapDataType dt, int elem_bytes, const void* ptr, uint64_t rows,
               uint64_t cols, uint32_t box_cols, uint32_t box_rows);
// Row-major K x N bf16 matrix (N % 64 == 0) seen as [N/64][K][64]: one box of (64, box_k, n_blocks) brings
// n_blocks 64-column blocks of a k-slab with a single copy, each block laid out as a separate 2-D box would be.
bool encode_b_blocks(CUtensorMap* tm, const void* ptr, uint64_t K, uint64_t N, uint32_t box_k, uint32_t n_blocks);

// Host-side dispatchers of the kernel families (defined next to their kernels).
ag_status gemm_skinny_dispatch(const void* A, const void* B_rowmajor, const ag_packed_weights* W, void* Cout, int M,
                               int N, int K, const ag_plan* plan, float* partial, int* sem, cudaStream_t stream,
                               const ag_group_desc* grp = nullptr);
ag_status gemm_pair_dispatch(const void* A, const void* B, const ag_packed_weights* W, void* Cout, int M, int N, int K,
                             const ag_plan* plan, cudaStream_t stream, const ag_group_desc* grp = nullptr);

}  // namespace ag
