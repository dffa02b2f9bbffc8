// Sharing-preserving destination block allocation (section 3.4.5 counts shared prefixes among what a switch
// must leave intact): live table entries that name the same source block get the same destination block; distinct source blocks get base, base+1, ... in the order of their
// first occurrence when the tables are read row by row. Three kernels after the demand scan:
//   mark    every live entry k (flat position off[s] + j) records its source block and atomicMin's k into
//           first[source block];
//   scan    exclusive prefix sum over "entry k is the first of its block" (one CTA, running carry, so the
//           numbering is the serial one), block total and capacity check;
//   assign  every entry takes base + scan[first entry of its block]; first entries also append the
//           (source, destination) pair to the compact list the migration kernel walks.

#include "remp_internal.h"

namespace remp {

constexpr int kThreads = 256;
constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(kThreads) dedupe_mark_kernel(const int32_t* __restrict__ block_tables,
                                                              int32_t num_seqs, int32_t max_blocks,
                                                              const int32_t* __restrict__ off, int64_t src_pool,
                                                              int32_t* __restrict__ first,
                                                              int32_t* __restrict__ entry_src,
                                                              uint32_t* __restrict__ err) {
    if (*reinterpret_cast<volatile uint32_t*>(err) & kErrFatalMask) return;
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = (int64_t)gridDim.x * (kThreads / 32);
    bool bad = false;
    for (int64_t s = (int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); s < num_seqs; s += nwarps) {
        const int32_t o0 = off[s], need = off[s + 1] - o0;
        const int32_t* row = block_tables + s * max_blocks;
        for (int32_t j = lane; j < need; j += 32) {
            int32_t sb = row[j];
            if (sb < 0 || sb >= src_pool) {
                bad = true;
                sb = -1;
            } else {
                atomicMin(first + sb, o0 + j);
            }
            entry_src[o0 + j] = sb;
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(err, kErrBadBlock);
}

__global__ void __launch_bounds__(kScanThreads) dedupe_scan_kernel(const int32_t* __restrict__ entry_src,
                                                                  const int32_t* __restrict__ first,
                                                                  const int32_t* __restrict__ num_entries,
                                                                  int32_t* __restrict__ excl,
                                                                  int32_t* __restrict__ total, int64_t avail_blocks,
                                                                  uint32_t* __restrict__ err) {
    if (*reinterpret_cast<volatile uint32_t*>(err) & kErrFatalMask) return;
    __shared__ int32_t warp_sum[kScanThreads / 32];
    __shared__ int32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int32_t n = *num_entries;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int32_t tile = 0; tile < n; tile += kScanThreads) {
        const int32_t k = tile + tid;
        int32_t flag = 0;
        if (k < n) {
            const int32_t sb = entry_src[k];
            flag = (sb < 0 || first[sb] == k) ? 1 : 0;  // an entry outside the pool gets a block of its own
        }
        int32_t incl = flag;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            int32_t v = warp_sum[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int32_t up = __shfl_up_sync(0xffffffffu, v, d);
                if (lane >= d) v += up;
            }
            warp_sum[lane] = v;
        }
        __syncthreads();
        const int32_t carry = carry_s;
        if (k < n) excl[k] = carry + (wid ? warp_sum[wid - 1] : 0) + incl - flag;
        __syncthreads();
        if (tid == kScanThreads - 1) carry_s = carry + warp_sum[kScanThreads / 32 - 1];
        __syncthreads();
    }
    if (tid == 0) {
        *total = carry_s;
        if ((int64_t)carry_s > avail_blocks) atomicOr(err, kErrCapacity);
    }
}

__global__ void __launch_bounds__(kThreads) dedupe_assign_kernel(int32_t num_seqs, int32_t max_blocks,
                                                                int32_t base_block, const int32_t* __restrict__ off,
                                                                const int32_t* __restrict__ entry_src,
                                                                const int32_t* __restrict__ first,
                                                                const int32_t* __restrict__ excl,
                                                                int32_t* __restrict__ dst_block_tables,
                                                                int4* __restrict__ pairs,
                                                                int32_t block_size,
                                                                const uint32_t* __restrict__ err) {
    if (*reinterpret_cast<const volatile uint32_t*>(err) & kErrFatalMask) return;
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t s = (int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); s < num_seqs; s += nwarps) {
        const int32_t o0 = off[s], need = off[s + 1] - o0;
        int32_t* out = dst_block_tables + s * max_blocks;
        for (int32_t j = lane; j < max_blocks; j += 32) {
            if (j < need) {
                const int32_t k = o0 + j, sb = entry_src[k];
                const int32_t f = sb >= 0 ? first[sb] : k;
                const int32_t db = base_block + excl[f];
                out[j] = db;
                if (f == k) pairs[excl[k]] = make_int4(sb, db, block_size, 0);  // a shared block counts as full
            } else {
                out[j] = -1;
            }
        }
    }
}

cudaError_t launch_dedupe(const int32_t* block_tables, int32_t num_seqs, int32_t max_blocks, int32_t base_block,
                          const int32_t* off, int64_t src_pool, int64_t avail_blocks, int32_t* first,
                          int32_t* entry_src, int32_t* excl, int32_t* dst_block_tables, int4* pairs, int32_t* total,
                          uint32_t* err, cudaStream_t stream, int32_t block_size) {
    if (num_seqs == 0 || max_blocks == 0) return cudaSuccess;
    // 0x7f7f7f7f is larger than any entry position (positions are checked to fit 31 bits)
    cudaError_t e = cudaMemsetAsync(first, 0x7f, (size_t)(src_pool > 0 ? src_pool : 1) * sizeof(int32_t), stream);
    if (e != cudaSuccess) return e;
    int64_t blocks = ((int64_t)num_seqs + kThreads / 32 - 1) / (kThreads / 32);
    const int grid = (int)(blocks < 65536 ? blocks : 65536);
    dedupe_mark_kernel<<<grid, kThreads, 0, stream>>>(block_tables, num_seqs, max_blocks, off, src_pool, first,
                                                      entry_src, err);
    dedupe_scan_kernel<<<1, kScanThreads, 0, stream>>>(entry_src, first, off + num_seqs, excl, total, avail_blocks, err);
    dedupe_assign_kernel<<<grid, kThreads, 0, stream>>>(num_seqs, max_blocks, base_block, off, entry_src, first, excl,
                                                        dst_block_tables, pairs, block_size, err);
    count_launch(3);
    return cudaGetLastError();
}

}  // namespace remp
