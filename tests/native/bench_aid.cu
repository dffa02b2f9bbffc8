// Bandwidth probe: plain sequential read, write and copy streams driven by the same scheduler as the migration
// kernel (persistent CTAs drawing tiles of eight 4 KiB chunks from a device counter, 16-byte streaming
// accesses). It answers "what can this device do when nothing is gathered or scattered", the yardstick the
// migration kernel's GB/s is read against besides a library copy.

#include "remp_internal.h"

namespace remp {
remp_status report_error(remp_status st, const char* msg);
}

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

extern "C" remp_status remp_probe_bandwidth(int32_t mode, const void* src, void* dst, int64_t bytes, uint32_t* scratch,
                                            int32_t ctas_per_sm, void* stream_) {
    if (mode < 0 || mode > 2 || bytes < 0 || bytes % 4096 != 0 || !scratch || (mode != 1 && !src) || (mode != 0 && !dst))
        return remp::report_error(REMP_ERR_INVALID_ARG, "mode 0..2, bytes a multiple of 4096, non-null buffers");
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (e == cudaSuccess) e = cudaMemsetAsync(scratch, 0, 2 * sizeof(uint32_t), stream);
    if (e != cudaSuccess) return remp::report_error(REMP_ERR_CUDA, cudaGetErrorString(e));
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
    remp::count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return remp::report_error(REMP_ERR_CUDA, cudaGetErrorString(e));
    return REMP_OK;
}
