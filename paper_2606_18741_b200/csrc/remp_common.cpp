// Shared host helpers of libremp: per-thread error text, launch counter, per-device memory pools.

#include <atomic>
#include <mutex>

#include "remp_internal.h"

namespace remp {

static thread_local std::string g_last_error;
static std::atomic<int64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
int64_t launch_count() { return g_launches.load(std::memory_order_relaxed); }

remp_status fail(remp_status st, const std::string& msg) {
    g_last_error = msg;
    return st;
}

remp_status report_error(remp_status st, const char* msg) { return fail(st, msg); }

remp_status cuda_fail(cudaError_t e, const char* what) {
    return fail(REMP_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

const char* last_error() { return g_last_error.c_str(); }

// Library-owned memory pools, one per device, created on first use. Plans take their scratch from them
// in stream order, and the pools keep freed scratch, so a switch costs no cudaMalloc.
static std::mutex g_pool_mu;
static cudaMemPool_t g_pools[64] = {};

remp_status device_pool(int device, cudaMemPool_t* out) {
    std::lock_guard<std::mutex> lock(g_pool_mu);
    if (device < 0 || device >= 64) return fail(REMP_ERR_INVALID_ARG, "device index out of range");
    if (!g_pools[device]) {
        cudaMemPoolProps props{};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        REMP_CUDA(cudaMemPoolCreate(&g_pools[device], &props));
        uint64_t keep = UINT64_MAX;  // never hand scratch back to the driver between switches
        REMP_CUDA(cudaMemPoolSetAttribute(g_pools[device], cudaMemPoolAttrReleaseThreshold, &keep));
    }
    *out = g_pools[device];
    return REMP_OK;
}

remp_status trim_pools() {
    std::lock_guard<std::mutex> lock(g_pool_mu);
    for (cudaMemPool_t pool : g_pools)
        if (pool) REMP_CUDA(cudaMemPoolTrimTo(pool, 0));
    return REMP_OK;
}

}  // namespace remp

extern "C" const char* remp_last_error(void) { return remp::last_error(); }
extern "C" remp_status remp_release_cached_memory(void) { return remp::trim_pools(); }
extern "C" int64_t remp_kernel_launch_count(void) { return remp::launch_count(); }
