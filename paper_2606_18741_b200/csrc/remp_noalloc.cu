// remp_remap_tables_noalloc: destination block allocation and block-table rewrite for callers that must not
// allocate device memory. Its only scratch - the per-sequence prefix offsets, the block total and the
// status word - lives in a fixed-size array inside the library image instead of a pool allocation.

#include <mutex>

#include "remp_internal.h"

namespace {

constexpr int kMaxSeqs = REMP_NOALLOC_MAX_SEQS;
// [0 .. num_seqs] exclusive prefix offsets | [kMaxSeqs+1] total | [kMaxSeqs+2] status word.
// Every GPU that loads the library holds these 256 KiB until the process exits.
static __device__ __align__(256) int32_t g_noalloc_scratch[kMaxSeqs + 4];

// The array's name is only a host-side handle; kernels need the device address, looked up once per device.
std::mutex g_mu;
int32_t* g_scratch_addr[64] = {};

remp_status scratch_for_current_device(int32_t** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return remp::report_error(REMP_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return remp::report_error(REMP_ERR_INVALID_ARG, "device index out of range");
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        int32_t* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return remp::report_error(REMP_ERR_CUDA, e != cudaSuccess ? cudaGetErrorString(e)
                                                                      : "cudaGetSymbolAddress returned a null address");
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return REMP_OK;
}

constexpr int kThreads = 256;

// The table remapper without the pair list: one warp per sequence writes base + off[s] + j for the live
// entries of row s and -1 for the padding; nothing when the scan recorded a fatal condition. Thread 0 of
// CTA 0 then hands the scan's total and status word to the caller.
__global__ void __launch_bounds__(kThreads) remap_tables_noalloc_kernel(int32_t num_seqs, int32_t max_blocks,
                                                                       int32_t base_block,
                                                                       const int32_t* __restrict__ off,
                                                                       const int32_t* __restrict__ total,
                                                                       const uint32_t* __restrict__ err,
                                                                       int32_t* __restrict__ dst_block_tables,
                                                                       int32_t* __restrict__ result) {
    const uint32_t status = *err;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        result[0] = *total;
        result[1] = (int32_t)status;
    }
    if (status & remp::kErrFatalMask) return;
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t s = (int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); s < num_seqs; s += nwarps) {
        const int32_t o0 = off[s], need = off[s + 1] - o0;
        int32_t* out = dst_block_tables + s * max_blocks;
        for (int32_t j = lane; j < max_blocks; j += 32) out[j] = j < need ? base_block + o0 + j : -1;
    }
}

}  // namespace

extern "C" remp_status remp_remap_tables_noalloc(const int32_t* seq_lens, int32_t num_seqs, int32_t max_blocks_per_seq,
                                                 int32_t block_size, int32_t base_block, int64_t capacity_blocks,
                                                 int32_t* dst_block_tables, int32_t* result, void* stream_) {
    if (num_seqs < 0 || max_blocks_per_seq < 0 || block_size < 1 || base_block < 0 || capacity_blocks < 0)
        return remp::report_error(REMP_ERR_INVALID_ARG, "negative size, block_size < 1 or negative capacity");
    if (num_seqs > kMaxSeqs)
        return remp::report_error(REMP_ERR_INVALID_ARG,
                                  "num_seqs exceeds REMP_NOALLOC_MAX_SEQS, the size of the built-in scratch array");
    if (!result || (num_seqs > 0 && (!seq_lens || (max_blocks_per_seq > 0 && !dst_block_tables))))
        return remp::report_error(REMP_ERR_INVALID_ARG, "null argument");
    int32_t* scratch = nullptr;
    if (remp_status st = scratch_for_current_device(&scratch)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int32_t* total = scratch + kMaxSeqs + 1;
    uint32_t* err = reinterpret_cast<uint32_t*>(scratch + kMaxSeqs + 2);
    // The array keeps what the previous call left: the total and the status word must start at zero
    // (the offsets [0 .. num_seqs] are all rewritten by the scan).
    cudaError_t e = cudaMemsetAsync(total, 0, 2 * sizeof(int32_t), stream);
    // ids are 32-bit: blocks at or beyond 2^31 - base_block cannot be named, so they do not count as capacity
    int64_t avail = capacity_blocks > base_block ? capacity_blocks - base_block : 0;
    if (avail > 0x7fffffffLL - base_block) avail = 0x7fffffffLL - base_block;
    if (e == cudaSuccess)
        e = remp::launch_demand_scan(seq_lens, num_seqs, block_size, max_blocks_per_seq, avail, scratch, total, err,
                                     stream);
    if (e == cudaSuccess) {
        int64_t blocks = ((int64_t)num_seqs + kThreads / 32 - 1) / (kThreads / 32);
        const int grid = (int)(blocks < 1 ? 1 : (blocks < 65536 ? blocks : 65536));
        remap_tables_noalloc_kernel<<<grid, kThreads, 0, stream>>>(num_seqs, max_blocks_per_seq, base_block, scratch,
                                                                   total, err, dst_block_tables, result);
        remp::count_launch();
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return remp::report_error(REMP_ERR_CUDA, cudaGetErrorString(e));
    return REMP_OK;
}
