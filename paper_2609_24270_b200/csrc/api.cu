// Small shared pieces of the C ABI: error strings, architecture check, launch accounting.
#include <stdio.h>
#include <string.h>

#include "internal.h"
#include "ptx.cuh"

namespace ag {
thread_local int g_last_cuda_error = 0;
std::atomic<unsigned long long> g_launch_count{0};

ag_status cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    cudaGetLastError();  // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? AG_ERR_NOMEM : AG_ERR_CUDA;
}

ag_status check_arch() {
    int dev = 0, major = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    return major == 10 ? AG_OK : AG_ERR_UNSUPPORTED_ARCH;
}
}  // namespace ag

// Host arithmetic only (no device is touched).  Candidates are the powers of two up to 32 that leave every split at
// least four k-slabs; the score of a candidate is (how evenly its units fill the SMs) x (share of a unit's time that is
// streaming): a unit costs about as much as 20 KB of weights on top of its own bytes, and without overlapping launches
// the longest list of ceil(units / SMs) units sets the time.
extern "C" int32_t ag_suggest_k_splits(int32_t N, int32_t K, int32_t sm_budget, int32_t overlapping_full_chip) {
    if (N <= 0 || K <= 0 || sm_budget <= 0) return 1;
    const long long tiles = (N + 127) / 128;
    const int n_slab = (K + 63) / 64;
    int best = 1;
    double best_score = -1.0;
    for (int ksp = 1; ksp <= 32; ksp *= 2) {
        const int per = (n_slab + ksp - 1) / ksp;
        if (ksp > 1 && (per < 4 || (long long)(ksp - 1) * per >= n_slab)) break;
        const double units = (double)(tiles * ksp), per_sm = units / sm_budget;
        const long long longest = (tiles * ksp + sm_budget - 1) / sm_budget;
        const double balance = overlapping_full_chip ? (per_sm < 1.0 ? per_sm : 1.0) : per_sm / (double)longest;
        const double unit_kb = 128.0 * per * 64.0 * 2.0 / 1024.0;
        const double score = balance * unit_kb / (unit_kb + 20.0);
        if (score > best_score + 1e-9) { best_score = score; best = ksp; }
    }
    return best;
}

extern "C" const char* ag_strerror(ag_status s) {
    switch (s) {
        case AG_OK: return "ok";
        case AG_ERR_ARG: return "bad argument";
        case AG_ERR_CUDA: return "CUDA call failed";
        case AG_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case AG_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case AG_ERR_UNMANNED_SM: return "an SM of the set never got a thread block";
        case AG_ERR_NOISY_PROBE: return "latency tiers could not be separated";
        case AG_ERR_STALE_AMAP: return "affinity map does not belong to this buffer";
        case AG_ERR_NOMEM: return "out of memory";
    }
    return "unknown status";
}

extern "C" int ag_last_cuda_error(void) { return ag::g_last_cuda_error; }
extern "C" uint64_t ag_kernel_launch_count(void) { return ag::g_launch_count.load(); }

// ---- bounded-wait self test ---------------------------------------------------------------------
// One thread waits on an mbarrier that nothing ever arrives at; the wait gives up after limit_ns and
// the kernel reports it, exactly as the persistent kernels do when a copy or an MMA never signals.
namespace ag {
__global__ void k_wait_probe(unsigned long long limit_ns, int* status, unsigned long long* waited_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        mbar_fence_init();
        const uint64_t t0 = globaltimer_ns();
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns);
        *waited_ns = globaltimer_ns() - t0;
        *status = ok ? (int)AG_OK : (int)AG_ERR_TIMEOUT;
    }
}
}  // namespace ag

extern "C" ag_status ag_wait_probe(uint64_t limit_ns, uint64_t* waited_ns) {
    if (limit_ns == 0 || limit_ns > 1000000000ull) return AG_ERR_ARG;  // at most one second
    ag_status st = ag::check_arch();
    if (st != AG_OK) return st;
    int* d_status = nullptr;
    unsigned long long* d_waited = nullptr;
    AG_CUDA(cudaMalloc(&d_status, sizeof(int)));
    cudaError_t e = cudaMalloc(&d_waited, sizeof(unsigned long long));
    int h_status = -1;
    unsigned long long h_waited = 0;
    if (e == cudaSuccess) {
        ag::k_wait_probe<<<1, 32>>>(limit_ns, d_status, d_waited);
        ag::count_launch();
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&h_status, d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(&h_waited, d_waited, sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    cudaFree(d_status);
    cudaFree(d_waited);
    if (e != cudaSuccess) return ag::cuda_fail(e);
    if (waited_ns) *waited_ns = h_waited;
    return (ag_status)h_status;
}

// ---- topology map on disk ---------------------------------------------------------------------
// Discovery takes a fraction of a second here but the paper budgets up to a minute per GPU; the map is a
// plain struct, so it can be kept in a file and reused by later processes on the same GPU.
static const char kTopoMagic[8] = {'A', 'G', 'T', 'O', 'P', 'O', '0', '1'};

extern "C" ag_status ag_topo_save(const ag_topo_map* map, const char* path) {
    if (!map || !path) return AG_ERR_ARG;
    FILE* f = fopen(path, "wb");
    if (!f) return AG_ERR_ARG;
    const bool ok = fwrite(kTopoMagic, 1, 8, f) == 8 && fwrite(map, sizeof *map, 1, f) == 1;
    return (fclose(f) == 0 && ok) ? AG_OK : AG_ERR_ARG;
}

extern "C" ag_status ag_topo_load(const char* path, ag_topo_map* map) {
    if (!map || !path) return AG_ERR_ARG;
    FILE* f = fopen(path, "rb");
    if (!f) return AG_ERR_ARG;
    char magic[8];
    ag_topo_map tmp;
    const bool ok = fread(magic, 1, 8, f) == 8 && memcmp(magic, kTopoMagic, 8) == 0 && fread(&tmp, sizeof tmp, 1, f) == 1 &&
                    fgetc(f) == EOF;
    fclose(f);
    if (!ok || tmp.n_sm <= 0 || tmp.n_sm > AG_MAX_SM || tmp.n_gpc < 0 || tmp.n_gpc > AG_MAX_GPC) return AG_ERR_ARG;
    int sum = 0;
    for (int s = 0; s < tmp.n_sm; ++s) {
        if (tmp.die[s] < 0 || tmp.die[s] >= AG_MAX_DIE || tmp.gpc[s] >= tmp.n_gpc) return AG_ERR_ARG;
        ++sum;
    }
    if (tmp.die_sm_count[0] + tmp.die_sm_count[1] != sum) return AG_ERR_ARG;
    *map = tmp;
    return AG_OK;
}
