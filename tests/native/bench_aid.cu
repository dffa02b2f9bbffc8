// Measuring aids of the benchmark (not part of the library, not part of the paper's method):
//   benchaid_probe_bandwidth  plain sequential read, write and copy streams driven by the same kind of scheduler
//                             as the migration kernel (persistent CTAs drawing tiles of eight 4 KiB chunks from
//                             a device counter, 16-byte streaming accesses): what the device does when nothing is
//                             gathered or scattered.
//   benchaid_switch_loop      a C loop over whole switches (remp_plan_create, remp_alloc_dst_blocks,
//                             remp_migrate_kv, remp_plan_destroy) through the library's C ABI, so that the cost
//                             of a small switch can be read without an interpreter between the calls.
// Built into its own shared object, which links against libremp.so.

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <chrono>
#include <vector>

#include "remp.h"

namespace {

__device__ __forceinline__ uint4 ld16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st16(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <int MODE>  // 0 read, 1 write, 2 copy
__global__ void __launch_bounds__(256) probe_kernel(const char* __restrict__ src, char* __restrict__ dst,
                                                   uint64_t nchunks, uint32_t* counter, uint32_t* sink) {
    __shared__ uint32_t next_tile[2];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) next_tile[0] = atomicAdd(counter, 1u);
    __syncthreads();
    uint32_t acc = 0;
    for (uint32_t buf = 0;; buf ^= 1) {
        const uint64_t t0 = (uint64_t)next_tile[buf] * 8;
        if (t0 >= nchunks) break;
        if (threadIdx.x == 0) next_tile[buf ^ 1] = atomicAdd(counter, 1u);
        const uint64_t w = t0 + warp;
        if (w < nchunks) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (MODE != 1)
                    v[u] = ld16(src + w * 4096 + (u * 32 + lane) * 16);
                else
                    v[u] = make_uint4((uint32_t)w, u, lane, 0);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (MODE != 0)
                    st16(dst + w * 4096 + (u * 32 + lane) * 16, v[u]);
                else
                    acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
            }
        }
        __syncthreads();
    }
    if (MODE == 0 && acc == 0x9e3779b9u) *sink = acc;  // keeps the loads alive
}

}  // namespace

// mode 0 reads src, 1 writes dst, 2 copies src to dst. src / dst: DEVICE, 16-byte aligned, `bytes` (a multiple of
// 4096) long; scratch: DEVICE, 2 x uint32 owned by the caller; ctas_per_sm 0 = 3. Only enqueues on `stream`.
// Returns 0 or a cudaError_t / -1 for bad arguments.
extern "C" int benchaid_probe_bandwidth(int32_t mode, const void* src, void* dst, int64_t bytes, uint32_t* scratch,
                                        int32_t ctas_per_sm, void* stream_) {
    if (mode < 0 || mode > 2 || bytes < 0 || bytes % 4096 != 0 || !scratch || (mode != 1 && !src) || (mode != 0 && !dst))
        return -1;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (e == cudaSuccess) e = cudaMemsetAsync(scratch, 0, 2 * sizeof(uint32_t), stream);
    if (e != cudaSuccess) return (int)e;
    const int grid = sms * (ctas_per_sm > 0 ? ctas_per_sm : 3);
    const uint64_t n = (uint64_t)bytes / 4096;
    const char* s = static_cast<const char*>(src);
    char* d = static_cast<char*>(dst);
    if (mode == 0)
        probe_kernel<0><<<grid, 256, 0, stream>>>(s, d, n, scratch, scratch + 1);
    else if (mode == 1)
        probe_kernel<1><<<grid, 256, 0, stream>>>(s, d, n, scratch, scratch + 1);
    else
        probe_kernel<2><<<grid, 256, 0, stream>>>(s, d, n, scratch, scratch + 1);
    return (int)cudaGetLastError();
}

// One transition of a topology chain, every argument as the library's calls take it.
typedef struct {
    const remp_topo* src;
    const remp_topo* dst;
    const remp_block_tables* tables;
    const int64_t* dst_capacity_blocks;
    int32_t* dst_block_tables;
    const remp_shard* src_shards;
    const remp_shard* dst_shards;
} benchaid_leg;

// Runs `steps` passes over the legs on `stream`; every switch is remp_plan_create + remp_alloc_dst_blocks (no host
// read-back) + remp_migrate_kv + remp_plan_destroy, or - with reuse_plans - only the middle two on plans made once.
// host_us: wall time of the enqueueing loop per switch; device_us: CUDA-event time per switch over the loop
// (the larger of the two bounds the switch rate). Returns 0, or the failing remp_status.
extern "C" int benchaid_switch_loop(const remp_model_shape* shape, const benchaid_leg* legs, int32_t n_legs,
                                    int32_t reuse_plans, int32_t steps, void* stream_, double* host_us,
                                    double* device_us) {
    if (!shape || !legs || n_legs < 1 || steps < 1 || !host_us || !device_us) return REMP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<remp_plan*> plans((size_t)n_legs, nullptr);
    int rc = REMP_OK;
    auto make = [&](int i) { return (int)remp_plan_create(legs[i].src, legs[i].dst, shape, legs[i].tables, &plans[i]); };
    auto run = [&](int i) {
        int st = remp_alloc_dst_blocks(plans[i], legs[i].dst_capacity_blocks, 0, legs[i].dst_block_tables, nullptr, stream);
        if (st == REMP_OK) st = remp_migrate_kv(plans[i], legs[i].src_shards, legs[i].dst_shards, stream);
        return st;
    };
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    for (int pass = 0; pass < 2 && rc == REMP_OK; ++pass) {  // pass 0 warms up (a tenth of the steps), pass 1 is timed
        const int n = pass == 0 ? (steps + 9) / 10 : steps;
        if (reuse_plans)
            for (int i = 0; i < n_legs && rc == REMP_OK; ++i)
                if (!plans[i]) rc = make(i);
        cudaStreamSynchronize(stream);
        const auto t0 = std::chrono::steady_clock::now();
        cudaEventRecord(e0, stream);
        for (int s = 0; s < n && rc == REMP_OK; ++s)
            for (int i = 0; i < n_legs && rc == REMP_OK; ++i) {
                if (!reuse_plans) rc = make(i);
                if (rc == REMP_OK) rc = run(i);
                if (!reuse_plans && plans[i]) {
                    remp_plan_destroy(plans[i]);  // scratch is released in stream order, behind the enqueued work
                    plans[i] = nullptr;
                }
            }
        cudaEventRecord(e1, stream);
        const auto t1 = std::chrono::steady_clock::now();
        cudaStreamSynchronize(stream);
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        *host_us = std::chrono::duration<double, std::micro>(t1 - t0).count() / ((double)n * n_legs);
        *device_us = (double)ms * 1e3 / ((double)n * n_legs);
    }
    for (int i = 0; i < n_legs; ++i)
        if (plans[i]) {
            if (rc == REMP_OK) rc = remp_plan_status(plans[i], stream);
            remp_plan_destroy(plans[i]);
        }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return rc;
}
