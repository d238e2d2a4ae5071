// Device-side pieces shared by the persistent kernels: joining the plan (which SM am I, is it
// planned, take its slot), and the source of work units (static per-SM list with adoption of
// unmanned lists, or dynamic pulls from the per-die queues).  Section 7.1.2 of the paper: one
// persistent block per SM that asks which SM it runs on and processes the tasks planned for it.
#pragma once
#include <stddef.h>

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
    unsigned int* claimed;  // ctrl->claimed[epoch & 1]: the claim flags of this launch
    int32_t* tile_owner;
    int32_t* tile_count;
    unsigned long long* unit_times;   // [n_units][2] start / end in ns of the global timer, or null (tracing off)
    int M, N, K;
    int b, n_units, n_sm;
    int tiles_n, k_splits, kslabs_total, kslabs_per_split;
    int static_assign;
    unsigned int epoch;
    unsigned long long wait_limit_ns;
    unsigned long long manned_wait_ns;   // how long a block on an unplanned SM stays to keep that SM occupied (wait_until_manned)
    int b_blocks;           // 1: tm_b is the 3-D [N/64][K][64] view of B (one copy per k-slab)
    int a_blocks;           // 1: tm_a is the 3-D [K/64][M][64] view of A (decode-shaped kernel: one copy per 8 k-slabs)
    const int4* quick;      // [n_sm]: {slot, offset of the SM's list in sm_q, its length, its first unit} (slot -1: unplanned)
};

__device__ __forceinline__ void report_timeout(const PersistParams& p, int role) {
    if (atomicCAS(&p.ctrl->status, 0, (int)AG_ERR_TIMEOUT) == 0) p.ctrl->status_info = (role << 16) | (int)smid();
}

// Dynamic mode: take the next index of a die's queue; the 64-bit head carries the epoch of the
// launch that last touched it, so it resets itself.  Returns -1 when the queue is drained.
// Once the head carries this launch's epoch a pop is one fetch-and-add (a compare-and-swap loop here made 74 SMs
// that pop every few microseconds spend most of their time retrying); only the first pops of a launch race to
// move the head to the new epoch.  The index may run past len by one per pop after the end: far from 2^32.
__device__ inline int pop_queue(unsigned long long* head, unsigned int epoch, int len) {
    unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(head);
    for (int tries = 0; tries < 100000; ++tries) {
        if ((unsigned int)(cur >> 32) == epoch) {
            const unsigned long long old = atomicAdd(head, 1ull);
            if ((unsigned int)(old >> 32) == epoch) {
                const unsigned int idx = (unsigned int)(old & 0xffffffffull);
                return idx < (unsigned int)max(len, 0) ? (int)idx : -1;
            }
            cur = old + 1;      // (a head of another epoch: launches of a dynamic plan never overlap, so this is not reached)
            continue;
        }
        const unsigned long long fresh = (unsigned long long)epoch << 32;
        const unsigned long long seen = atomicCAS(head, cur, fresh);
        cur = seen == cur ? fresh : seen;
    }
    return -1;
}

// True when a block of this launch has taken the slot.  (A later epoch in the flag can only come from a launch
// that started after this one had manned all its SMs; it counts as taken, so that nobody ever waits on it.)
__device__ __forceinline__ bool epoch_reached(unsigned int flag, unsigned int epoch) { return (int)(flag - epoch) >= 0; }
__device__ __forceinline__ bool slot_taken(const PersistParams& p, int i) {
    return epoch_reached(*reinterpret_cast<volatile unsigned int*>(&p.claimed[i]), p.epoch);
}

// A block on an unplanned SM stays resident until every planned SM has a block (at most ~40 us; with overlapping
// launches on part of the chip until the launch before has left the planned SMs, bounded like every other wait),
// so that blocks still being placed can only land on SMs that have none yet.  Called by every thread.
__device__ inline void wait_until_manned(const PersistParams& p) {
    const uint64_t t0 = globaltimer_ns();
    while (true) {
        int ok = 1;
        for (int i = threadIdx.x; i < p.b; i += blockDim.x) ok &= slot_taken(p, i) ? 1 : 0;
        if (__syncthreads_and(ok)) break;
        if (globaltimer_ns() - t0 > p.manned_wait_ns) break;
        __nanosleep(200);
    }
}

// Called by every thread of the block.  Returns the plan slot of this block's SM, or -1 if the
// block has nothing to do (SM not in the plan, or its slot already taken by another block).
__device__ inline int join_plan(const PersistParams& p, int* s_member) {
    const PlanLayout lay{p.b, p.n_units, p.n_sm};
    const int slot = p.image[lay.smid_to_slot() + (int)smid()];
    if (slot < 0) {
        wait_until_manned(p);
        return -1;
    }
    if (threadIdx.x == 0) *s_member = atomicMax(&p.claimed[slot], p.epoch) < p.epoch;
    __syncthreads();
    return *s_member ? slot : -1;
}

// Source of work units for one block.  Warp-collective: every lane of the scheduler warp holds the
// same state and calls the functions together; atomics are done by lane 0 and broadcast.  A static list
// is read 32 entries at a time (lane l keeps entry l of the current run), so that handing out a unit
// costs no memory access.
struct UnitSource {
    const PersistParams& p;
    PlanLayout lay;
    int idx, list_off, list_len, scan, dyn_die;
    int cache, first;

    // off / len / first_unit: the SM's list as found in PersistParams::quick (saves two dependent loads), or -1
    __device__ UnitSource(const PersistParams& pp, int slot, int lane, int off = -1, int len = -1, int first_unit = -1)
        : p(pp), lay{pp.b, pp.n_units, pp.n_sm} {
        idx = 0;
        if (off >= 0) {
            list_off = off;
            list_len = len;
        } else {
            list_off = p.image[lay.sm_q_off() + slot];
            list_len = p.image[lay.sm_q_off() + slot + 1] - list_off;
        }
        first = first_unit;
        scan = 0;
        dyn_die = p.static_assign ? 0 : p.image[lay.sm_die() + slot];
        fill(lane);
    }
    __device__ void fill(int lane) {
        const int i = (idx & ~31) + lane;
        cache = (p.static_assign && i < list_len) ? p.image[lay.sm_q() + list_off + i] : -1;
    }
    // static lists: next unit of the list in hand, -1 when it is finished
    __device__ int next_listed(int lane) {
        if (idx >= list_len) return -1;
        int u;
        if (idx == 0 && first >= 0) u = first;   // known before the list itself has arrived
        else u = __shfl_sync(0xffffffffu, cache, idx & 31);
        ++idx;
        if ((idx & 31) == 0 && idx < list_len) fill(lane);
        return u;
    }
    // static lists: look for a planned SM that never got a block and take its list.  The claim flags of all slots
    // are fetched with independent loads (32 per lane-load, all in flight together: one L2 round trip instead of
    // one per flag).  False when every list has an owner.
    __device__ bool adopt(int lane) {
        for (int round = 0; round <= p.b; ++round) {   // every round settles one slot: b + 1 rounds always suffice
            unsigned int v[AG_MAX_SM / 32];
#pragma unroll
            for (int j = 0; j < AG_MAX_SM / 32; ++j) {
                const int i = j * 32 + lane;
                v[j] = (i >= scan && i < p.b) ? *reinterpret_cast<volatile unsigned int*>(&p.claimed[i]) : p.epoch;
            }
            int cand = -1;
#pragma unroll
            for (int j = 0; j < AG_MAX_SM / 32; ++j) {
                const unsigned m = __ballot_sync(0xffffffffu, !epoch_reached(v[j], p.epoch));
                if (m && cand < 0) cand = j * 32 + __ffs(m) - 1;
            }
            if (cand < 0) {
                scan = p.b;
                return false;
            }
            scan = cand;   // slots below cand have owners; cand itself is looked at again if the claim below fails
            int got = 0;
            if (lane == 0) got = atomicMax(&p.claimed[cand], p.epoch) < p.epoch;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (got) {
                list_off = p.image[lay.sm_q_off() + cand];
                list_len = p.image[lay.sm_q_off() + cand + 1] - list_off;
                idx = 0;
                first = -1;
                fill(lane);
                if (lane == 0) atomicAdd(&p.ctrl->adopted, 1u);
                return true;
            }
        }
        return false;
    }
    // next unit id, or -1 when there is nothing left for this block
    __device__ int next(int lane) {
        if (p.static_assign) {
            while (true) {
                const int u = next_listed(lane);
                if (u >= 0) return u;
                if (!adopt(lane)) return -1;
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

// A launch carries its epoch in the kernel parameters, so a launch recorded into a CUDA graph would repeat
// an old epoch on every replay and no block would join the plan: calls on a capturing stream are refused.
inline ag_status refuse_capture(cudaStream_t stream) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    AG_CUDA(cudaStreamIsCapturing(stream, &cs));
    return cs == cudaStreamCaptureStatusNone ? AG_OK : AG_ERR_ARG;
}

// Epochs are 32-bit and only ever grow: shortly before they would wrap (some 36 hours of back-to-back 30 us
// launches) the claim flags and queue heads are wiped on the stream and counting starts again.
inline ag_status renew_epochs_if_needed(const ag_plan* plan, cudaStream_t stream) {
    if (plan->epoch < 0xFFFFFF00u) return AG_OK;
    AG_CUDA(cudaMemsetAsync(plan->d_ctrl, 0, sizeof(PlanCtrl), stream));
    plan->epoch = 0;
    return AG_OK;
}

// Fills the launch parameters every persistent kernel needs from a plan (host) and takes the next epoch.
// Call launch_failed() if the launch does not happen after all.
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
    gp.claimed = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(plan->d_ctrl) + offsetof(PlanCtrl, claimed)) +
                 (size_t)AG_MAX_SM * (gp.epoch & 1u);
    gp.wait_limit_ns = kWaitLimitNs;
    gp.manned_wait_ns = 40000ull;
    gp.b_blocks = 0;
    gp.a_blocks = 0;
    gp.quick = plan->d_quick;
    return gp;
}
// The launch that make_persist_params prepared did not happen: give its epoch back, so that ag_last_status
// keeps describing the last launch that did run.
inline ag_status launch_failed(const ag_plan* plan, cudaError_t e) {
    --plan->epoch;
    return cuda_fail(e);
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
// Row-major rows x K bf16 matrix (K % 64 == 0) seen as [K/64][rows][64]: one box of (64, box_rows, n_slabs) brings
// n_slabs consecutive k-slabs of box_rows rows with a single copy, each slab laid out as a separate 2-D box would be.
bool encode_a_slabs(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t K, uint32_t box_rows, uint32_t n_slabs);

// Host-side dispatchers of the kernel families (defined next to their kernels).
// Plans that the decode-shaped (weight-streaming) kernel runs: 128-column units with at most 64 activation rows, or
// 128 rows when the policy says so (128 x 128 is also a tile of the dense one-block kernel).
inline bool is_decode_shaped(const ag_plan* plan) {
    const int32_t* h = plan->header;
    return h[H_TILE_N] == 128 && (h[H_TILE_M] <= 64 || (h[H_TILE_M] == 128 && plan->policy.decode_shaped));
}
// Stages (of 32 KB from memory each) of the streaming kernels' copy ring that a launch uses.  A bare copy ring on all 148
// SMs reads 7.38 TB/s with 3 or 4 stages per SM, 7.22 with 5, 7.16 with 6, and with 6 only 6.65 TB/s once the consumer holds
// a stage for 0.3 us as the MMA path does, while 4 stages lose nothing to that hold: beyond about 20 MB in flight on the
// chip the memory system is oversubscribed.  On half or a quarter of the SMs a block's rate grows with the bytes it keeps
// in flight.  policy.ring_stages > 0 overrides; otherwise `by_sm_count` selects 20 MiB shared by the plan's SMs (attention
// decode, whose launches last long enough to reach the steady state: 4 stages on the full chip read 3-7 % more than 6), or
// all stages (the decode-shaped GEMM, whose 20-microsecond launches gain more from a deep ring while they fill).
inline int ring_stages_for(const ag_plan* plan, int max_stages, int min_stages, bool even, bool by_sm_count) {
    int s = plan->policy.ring_stages;
    if (s <= 0) s = by_sm_count ? 640 / std::max(1, plan->lay.b) : max_stages;
    s = std::max(min_stages, std::min(max_stages, s));
    if (even && (s & 1)) s = s + 1 <= max_stages ? s + 1 : s - 1;
    return s;
}
ag_status gemm_skinny_dispatch(const void* A, const void* B_rowmajor, const ag_packed_weights* W, void* Cout, int M,
                               int N, int K, const ag_plan* plan, float* partial, cudaStream_t stream,
                               const ag_group_desc* grp = nullptr);
ag_status gemm_pair_dispatch(const void* A, const void* B, const ag_packed_weights* W, void* Cout, int M, int N, int K,
                             const ag_plan* plan, cudaStream_t stream, const ag_group_desc* grp = nullptr);

}  // namespace ag
