// gemm_persistent: persistent, warp-specialised BF16 GEMM for sm_100a whose thread blocks are
// pinned to the physical SMs of a plan (Section 7.1.2 of the paper: one persistent block per
// SM, each block reads which SM it runs on and processes the task list planned for that SM).
//
// One block per SM (the shared-memory footprint forbids a second one).  A block that lands
// on an SM outside the plan leaves; a member takes its slot and loops over its work units:
//   warp 0  (one lane)  scheduler + TMA producer: next unit -> ring, A/B k-slabs -> smem ring
//   warp 1  (one lane)  tcgen05.mma issuer, accumulators in tensor memory (two buffers)
//   warps 2-5           epilogue: tcgen05.ld -> registers -> swizzled smem -> TMA store
// Operands: A row-major (K-major) and B row-major (N-major) are both consumed in place; the
// MMA descriptors describe B as an MN-major operand, so no transpose pass exists.
#include <string.h>

#include <mutex>

#include "persist.cuh"

namespace ag {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kEpiBufBytes = 32 * 32 * 4;
// A warp gets only about two bulk copies in flight (measured), i.e. one stage (its A and its B box): the stages are
// filled by D_NPROD warps in turn, so that all of them can be in flight together.
constexpr int D_NPROD = 4;
constexpr int D_THREADS = (2 + kEpiWarps + D_NPROD) * 32;   // scheduler, MMA issuer, epilogue warps, copy warps

template <int BN>
struct Cfg {
    static constexpr int a_bytes = BM * BK * 2;
    static constexpr int b_bytes = BK * BN * 2;
    static constexpr int stage_bytes = a_bytes + b_bytes;
    static constexpr int epi_bytes = kEpiWarps * 2 * kEpiBufBytes;
    static constexpr int bar_bytes = 1024;
    static constexpr int budget = 227 * 1024 - 1024 /*alignment slack*/ - epi_bytes - bar_bytes;
    static constexpr int stages = budget / stage_bytes > 8 ? 8 : budget / stage_bytes;
    static constexpr int smem_bytes = stages * stage_bytes + epi_bytes + bar_bytes + 1024;
    static constexpr int tmem_cols = 2 * BN < 32 ? 32 : 2 * BN;  // power of two for BN in {64,128,256}
};

struct SharedCtl {
    uint64_t full[8];
    uint64_t empty[8];
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

template <int BN>
__global__ void __launch_bounds__(D_THREADS, 1)
k_gemm_persistent(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_c, const PersistParams p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t s_stage = base;
    const uint32_t s_epi = base + C::stages * C::stage_bytes;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + C::stages * C::stage_bytes + C::epi_bytes);
    volatile int* abort_flag = &ctl->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int my_sm = (int)smid();
    if (tid == 0) ctl->abort_flag = 0;
    const int slot = join_plan(p, &ctl->member);
    if (slot < 0) return;

    if (tid == 0) {
        for (int i = 0; i < C::stages; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), kEpiWarps);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&ctl->sched_full[i]), 1);
            mbar_init(smem_u32(&ctl->sched_empty[i]), 1 + kEpiWarps + D_NPROD);
        }
        mbar_init(smem_u32(&ctl->mma_drain), 1);
        mbar_fence_init();
        prefetch_tmap(&tm_a);
        prefetch_tmap(&tm_b);
        prefetch_tmap(&tm_c);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), C::tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const uint64_t limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------ scheduler (warp-collective): hands the unit ids to the other roles
        UnitSource src(p, slot, lane);
        int ok = 1;
        for (uint32_t it = 0; ok; ++it) {
            const int u = src.next(lane);
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
        // ------------------------------------------------ copies: warp pw fills the stages pw, pw + D_NPROD, ... of the block's run
        if (lane == 0) {
            const int pw = warp - (2 + kEpiWarps);
            uint32_t q_run = 0;      // stages before the current unit
            bool ok = true;
            for (uint32_t it = 0; ok; ++it) {
                const int r = it % kRing;
                if (!mbar_wait_idle(smem_u32(&ctl->sched_full[r]), (it / kRing) & 1, abort_flag, limit)) {
                    report_timeout(p, 8);
                    break;
                }
                const int u = ctl->ring[r];
                mbar_arrive(smem_u32(&ctl->sched_empty[r]));
                if (u < 0) break;
                const int ks = u % p.k_splits, t = u / p.k_splits;
                const int tm = t / p.tiles_n, tn = t % p.tiles_n;
                const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
                const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
                const int n = s1 - s0;
                const int i0 = (pw + D_NPROD - (int)(q_run % D_NPROD)) % D_NPROD;
                uint32_t st = (q_run + i0) % C::stages, ph = (((q_run + i0) / C::stages) & 1) ^ 1;   // stage, parity of "stage is free"
                for (int i = i0; i < n; i += D_NPROD) {
                    const int s = s0 + i;
                    if (!mbar_wait(smem_u32(&ctl->empty[st]), ph, abort_flag, limit)) {
                        report_timeout(p, 2);
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&ctl->full[st]);
                    const uint32_t sa = s_stage + st * C::stage_bytes, sb = sa + C::a_bytes;
                    mbar_expect_tx(bar, C::stage_bytes);
                    tma_load_2d(sa, &tm_a, bar, s * BK, tm * BM);
                    if (p.b_blocks) {
                        // one copy for all 64-column blocks of the slab (B seen as [N/64][K][64])
                        tma_load_3d(sb, &tm_b, bar, 0, s * BK, tn * (BN / 64));
                    } else {
#pragma unroll
                        for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * (BK * 128), &tm_b, bar, tn * BN + j * 64, s * BK);
                    }
                    st += D_NPROD;
                    while (st >= (uint32_t)C::stages) { st -= C::stages; ph ^= 1; }
                }
                q_run += (uint32_t)n;
            }
            if (!ok) {
                // gave up: linger (bounded) so that copies already in flight land before the block leaves
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer: the warp runs the loop converged, one elected lane issues (see elect_one)
        {
            constexpr uint32_t idesc = make_idesc_bf16(BM, BN, 0, 1);
            // descriptors without their start address.  A: K-major, 128-byte swizzle, 8-row groups 1024 B apart.
            // B: N-major, 128-byte swizzle: 64-column blocks 8 KB apart (LBO), 8-k groups 1 KB apart (SBO).
            const uint64_t da_t = make_smem_desc(0, 16, 1024, 2);
            const uint64_t db_t = make_smem_desc(0, BK * 128, 1024, 2);
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
                const int ks = u % p.k_splits;
                const int s0 = min(p.kslabs_total, ks * p.kslabs_per_split);
                const int s1 = min(p.kslabs_total, (ks + 1) * p.kslabs_per_split);
                const uint32_t acc = tile_it & 1;
                if (!mbar_wait_all(smem_u32(&ctl->tmem_empty[acc]), ((tile_it >> 1) & 1) ^ 1, abort_flag, limit)) {
                    if (lane == 0) report_timeout(p, 4);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int i = 0, n = s1 - s0; i < n; ++i) {
                    if (!mbar_wait_all(full0 + st * 8, ph, abort_flag, limit)) {
                        if (lane == 0) report_timeout(p, 5);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = s_stage + st * C::stage_bytes;
                    const uint64_t da = da_t | (uint64_t)(sa >> 4);
                    const uint64_t db = db_t | (uint64_t)((sa + C::a_bytes) >> 4);
                    if (elect_one()) {
                        tc_mma_f16(d_tmem, da, db, idesc, i > 0 ? 1u : 0u);
#pragma unroll
                        for (int k4 = 1; k4 < BK / 16; ++k4) tc_mma_f16(d_tmem, da + k4 * 2, db + k4 * 128, idesc, 1u);
                        tc_commit(empty0 + st * 8);  // slot reusable once these MMAs have read it
                    }
                    __syncwarp();
                    if (++st == (uint32_t)C::stages) { st = 0; ph ^= 1; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit(smem_u32(&ctl->tmem_full[acc]));
                __syncwarp();
                ++tile_it;
            }
            __syncwarp();
            if (*abort_flag) {
                // let issued MMAs retire before tensor memory is released
                if (elect_one()) {
                    tc_commit(smem_u32(&ctl->mma_drain));
                    int dummy = 0;
                    mbar_wait(smem_u32(&ctl->mma_drain), 0, &dummy, 2000000ull);
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------ epilogue warps
        const int q = warp & 3;  // tensor-memory lane quadrant this warp may read
        const uint32_t buf0 = s_epi + (warp - 2) * 2 * kEpiBufBytes;
        const bool reduce = p.k_splits > 1;
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
            const int t = u / p.k_splits;
            const int tm = t / p.tiles_n, tn = t % p.tiles_n;
            const uint32_t acc = tile_it & 1;
            if (!mbar_wait_warp(smem_u32(&ctl->tmem_full[acc]), (tile_it >> 1) & 1, abort_flag, limit)) {
                if (lane == 0) report_timeout(p, 7);
                break;
            }
            tc_fence_after();
            const int row0 = tm * BM + q * 32;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c, ++chunk_it) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c * 32, v);
                tmem_ld_wait();
                const uint32_t buf = buf0 + (chunk_it & 1) * kEpiBufBytes;
                if (lane == 0) bulk_wait_read<1>();  // the store that last used this buffer has read it
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
                    const int x = tn * BN + c * 32;
                    if (x < p.N && row0 < p.M) {
                        if (reduce) tma_reduce_add_2d(&tm_c, buf, x, row0);
                        else tma_store_2d(&tm_c, buf, x, row0);
                    }
                    bulk_commit();
                }
            }
            // accumulator fully read: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
                if (q == 0) {
                    p.tile_owner[u] = my_sm;
                    if (p.unit_times) p.unit_times[2 * u + 1] = globaltimer_ns();
                    atomicAdd(&p.tile_count[u], 1);
                }
            }
            ++tile_it;
        }
        if (lane == 0) bulk_wait<0>();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

bool encode_2d(CUtensorMap* tm, CUtensorMapDataType dt, int elem_bytes, const void* ptr, uint64_t rows,
               uint64_t cols, uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_b_blocks(CUtensorMap* tm, const void* ptr, uint64_t K, uint64_t N, uint32_t box_k, uint32_t n_blocks) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc || (N % 64)) return false;
    cuuint64_t dims[3] = {64, K, N / 64};
    cuuint64_t strides[2] = {N * 2, 128};
    cuuint32_t box[3] = {64, box_k, n_blocks};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_a_slabs(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t K, uint32_t box_rows, uint32_t n_slabs) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc || (K % 64)) return false;
    cuuint64_t dims[3] = {64, rows, K / 64};
    cuuint64_t strides[2] = {K * 2, 128};
    cuuint32_t box[3] = {64, box_rows, n_slabs};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
static ag_status launch(const ag_plan* plan, const PersistParams& gp, cudaStream_t stream) {
    using C = Cfg<BN>;
    static std::atomic<unsigned long long> attr_done{0};
    const cudaError_t attr_err = once_per_device(attr_done, [] {
        return cudaFuncSetAttribute(k_gemm_persistent<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::smem_bytes);
    });
    if (attr_err != cudaSuccess) return launch_failed(plan, attr_err);
    k_gemm_persistent<BN><<<plan->grid_blocks > 0 ? plan->grid_blocks : plan->lay.n_sm, D_THREADS, C::smem_bytes, stream>>>(plan->tm_a, plan->tm_b, plan->tm_c, gp);
    const cudaError_t le = cudaGetLastError();
    if (le != cudaSuccess) return launch_failed(plan, le);
    count_launch();
    return AG_OK;
}

}  // namespace ag

using namespace ag;

extern "C" ag_status gemm_persistent(const void* A, const void* B, void* Cout, int M, int N, int K,
                                     const ag_plan* plan, void* cuda_stream) {
    if (!A || !B || !Cout || !plan) return AG_ERR_ARG;
    const int32_t* h = plan->header;
    if (is_decode_shaped(plan))  // weights on the MMA's M side, split-K through the plan's scratch
        return gemm_skinny_dispatch(A, B, nullptr, Cout, M, N, K, plan, plan->d_partial,
                                    reinterpret_cast<cudaStream_t>(cuda_stream));
    if (M != h[H_M] || N != h[H_N] || K != h[H_K]) return AG_ERR_ARG;
    if (h[H_TILE_M] == 256)  // 256 x 256 units: pairs of blocks, full-chip plans only
        return gemm_pair_dispatch(A, B, nullptr, Cout, M, N, K, plan, reinterpret_cast<cudaStream_t>(cuda_stream));
    if (h[H_TILE_M] != BM || (h[H_TILE_N] != 64 && h[H_TILE_N] != 128 && h[H_TILE_N] != 256)) return AG_ERR_ARG;
    if (plan->policy.k_unit != BK) return AG_ERR_ARG;
    if ((K % 8) || (N % 8)) return AG_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)Cout) & 15u) return AG_ERR_ARG;
    ag_status st = check_arch();
    if (st != AG_OK) return st;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if ((st = refuse_capture(stream)) != AG_OK) return st;
    if ((st = renew_epochs_if_needed(plan, stream)) != AG_OK) return st;
    int dev = 0, n_sm = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (n_sm != plan->lay.n_sm) return AG_ERR_ARG;
    const int BN = h[H_TILE_N];
    if (plan->tm_a_ptr != A || plan->tm_b_ptr != B || plan->tm_c_ptr != Cout) {
        if (!encode_2d(&plan->tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, M, K, BK, BM)) return AG_ERR_CUDA;
        if (N % 64 == 0) {
            if (!encode_b_blocks(&plan->tm_b, B, K, N, BK, BN / 64)) return AG_ERR_CUDA;
        } else if (!encode_2d(&plan->tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, B, K, N, 64, BK)) {
            return AG_ERR_CUDA;
        }
        if (!encode_2d(&plan->tm_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Cout, M, N, 32, 32)) return AG_ERR_CUDA;
        plan->tm_a_ptr = A; plan->tm_b_ptr = B; plan->tm_c_ptr = Cout;
    }
    if (h[H_KSPLITS] > 1) AG_CUDA(cudaMemsetAsync(Cout, 0, sizeof(float) * (size_t)M * (size_t)N, stream));
    PersistParams gp = make_persist_params(plan, M, N, K);
    gp.b_blocks = (N % 64 == 0) ? 1 : 0;
    if (BN == 256) return launch<256>(plan, gp, stream);
    if (BN == 128) return launch<128>(plan, gp, stream);
    return launch<64>(plan, gp, stream);
}
