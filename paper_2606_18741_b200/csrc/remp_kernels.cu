// Device kernels of libremp for sm_100a: block-demand prefix scan, block-table remapper, and the
// KV migration (gather/scatter copy) kernel.

#include "remp_internal.h"

namespace remp {

// ---------------------------------------------------------------------------------------------
// K1: demand[s] = ceil(len[s] / block_size); off = exclusive prefix sum; total; capacity check.
// One CTA walks the sequences in tiles of kScanThreads with a running carry, so the result is the plain
// serial sum in sequence order and needs no inter-CTA communication.
// ---------------------------------------------------------------------------------------------
constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(kScanThreads) demand_scan_kernel(const int32_t* __restrict__ seq_lens,
                                                                  int32_t num_seqs, int32_t block_size,
                                                                  int32_t max_blocks, int64_t avail_blocks,
                                                                  int32_t* __restrict__ off,
                                                                  int32_t* __restrict__ total,
                                                                  uint32_t* __restrict__ err) {
    __shared__ long long warp_sum[kScanThreads / 32];
    __shared__ long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    uint32_t bad = 0;
    for (int32_t tile = 0; tile < num_seqs; tile += kScanThreads) {
        const int32_t s = tile + tid;
        long long need = 0;
        if (s < num_seqs) {
            const int32_t len = seq_lens[s];
            if (len < 0) {
                bad |= kErrBadLength;
            } else {
                need = ((long long)len + block_size - 1) / block_size;
                if (need > max_blocks) {
                    bad |= kErrBadLength;
                    need = 0;
                }
            }
        }
        long long incl = need;  // inclusive scan inside the warp
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const long long up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            long long v = warp_sum[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const long long up = __shfl_up_sync(0xffffffffu, v, d);
                if (lane >= d) v += up;
            }
            warp_sum[lane] = v;  // inclusive over warps
        }
        __syncthreads();
        const long long carry = carry_s;
        const long long before = carry + (wid ? warp_sum[wid - 1] : 0) + incl - need;
        if (s < num_seqs) off[s] = before > 0x7fffffffLL ? 0x7fffffff : (int32_t)before;
        __syncthreads();
        if (tid == kScanThreads - 1) carry_s = carry + warp_sum[kScanThreads / 32 - 1];
        __syncthreads();
    }
    const long long sum = carry_s;
    if (sum > 0x7fffffffLL) bad |= kErrOverflow;
    if (tid == 0) {
        if (sum > avail_blocks) bad |= kErrCapacity;
        off[num_seqs] = sum > 0x7fffffffLL ? 0x7fffffff : (int32_t)sum;
        *total = (bad & kErrOverflow) ? 0 : (int32_t)sum;
    }
    if (bad) atomicOr(err, bad);
}

// ---------------------------------------------------------------------------------------------
// K2: one warp per sequence. dst_bt[s][j] = base + off[s] + j for live entries, -1 for padding; the
// flat pair list pairs[off[s] + j] = (source block, destination block) drives the migration kernel.
// Writes nothing when the scan recorded a fatal condition (capacity, bad length, overflow).
// ---------------------------------------------------------------------------------------------
constexpr int kRemapThreads = 256;

__global__ void __launch_bounds__(kRemapThreads) remap_tables_kernel(const int32_t* __restrict__ block_tables,
                                                                    int32_t num_seqs, int32_t max_blocks,
                                                                    int32_t base_block,
                                                                    const int32_t* __restrict__ off,
                                                                    int32_t* __restrict__ dst_block_tables,
                                                                    int2* __restrict__ pairs,
                                                                    uint32_t* __restrict__ err) {
    if (*reinterpret_cast<volatile uint32_t*>(err) & kErrFatalMask) return;
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_cta = kRemapThreads / 32;
    const int64_t nwarps = (int64_t)gridDim.x * warps_per_cta;
    bool bad = false;
    for (int64_t s = (int64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5); s < num_seqs; s += nwarps) {
        int32_t o0 = 0, o1 = 0;
        if (lane == 0) {
            o0 = off[s];
            o1 = off[s + 1];
        }
        o0 = __shfl_sync(0xffffffffu, o0, 0);
        o1 = __shfl_sync(0xffffffffu, o1, 0);
        const int32_t need = o1 - o0;
        const int32_t* row = block_tables + s * max_blocks;
        int32_t* out = dst_block_tables + s * max_blocks;
        for (int32_t j = lane; j < max_blocks; j += 32) {
            if (j < need) {
                int32_t sb = row[j];
                const int32_t db = base_block + o0 + j;
                if (sb < 0) {
                    bad = true;
                    sb = -1;
                }
                out[j] = db;
                pairs[o0 + j] = make_int2(sb, db);
            } else {
                out[j] = -1;
            }
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(err, kErrBadBlock);
}

// ---------------------------------------------------------------------------------------------
// K3, register-copy variant. Work item w = chunk `ch` of run `i` of live block `k` of destination
// plane `g`; w increases along destination addresses, and consecutive warps of the grid take
// consecutive items, so at any moment the whole GPU writes one narrow window of one destination plane
// and reads one source plane (TLB- and DRAM-page friendly). A warp moves one chunk per iteration with
// 16-byte streaming loads and stores, all loads of the chunk in flight before the first store.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x),
                 "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

__device__ __forceinline__ Seg ld_seg(const Seg* p) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
    const uint2 b = __ldg(reinterpret_cast<const uint2*>(p) + 2);
    Seg s;
    s.base = ((uint64_t)a.y << 32) | a.x;
    s.bstride = (int64_t)(((uint64_t)a.w << 32) | a.z);
    s.nblocks = ((uint64_t)b.y << 32) | b.x;
    s.pad = 0;
    return s;
}

constexpr int kCopyThreads = 256;

template <int U>  // 16-byte vectors per lane per chunk: chunk = 512 * U bytes
__global__ void __launch_bounds__(kCopyThreads) migrate_regcopy_kernel(const MigrateParams p) {
    if (*reinterpret_cast<volatile uint32_t*>(p.err) & kErrFatalMask) return;
    const uint32_t nb = (uint32_t)*p.total;
    const uint32_t per_block = p.n_sub * p.nchunk;
    const uint32_t per_plane = nb * per_block;
    const uint64_t n_items = (uint64_t)per_plane * p.n_groups;  // < 2^32, checked on the host
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t warps = (uint64_t)gridDim.x * (kCopyThreads / 32);
    bool bad = false;
    for (uint64_t w64 = (uint64_t)blockIdx.x * (kCopyThreads / 32) + (threadIdx.x >> 5); w64 < n_items; w64 += warps) {
        const uint32_t w = (uint32_t)w64;
        const uint32_t g = w / per_plane, q = w - g * per_plane;
        const uint32_t k = q / per_block, r = q - k * per_block;
        const uint32_t i = r / p.nchunk, ch = r - i * p.nchunk;
        const uint32_t d = g * p.n_sub + i;
        const int2 pr = __ldg(p.pairs + k);
        const Seg ss = ld_seg(p.src_seg + d);
        const uint32_t off = ch * p.chunk_bytes;
        const uint32_t len = min(p.chunk_bytes, p.run_bytes - off);
        if ((uint64_t)(uint32_t)pr.x >= ss.nblocks) {  // also catches entries the remapper marked -1
            bad = true;
            continue;
        }
        const char* sp = reinterpret_cast<const char*>(ss.base + (int64_t)pr.x * ss.bstride + off);
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t o = (u * 32 + lane) * 16;
            if (o < len) v[u] = ld_stream(sp + o);
        }
        for (uint32_t rr = 0; rr < p.rep; ++rr) {
            const Seg ds = ld_seg(p.dst_seg + (uint64_t)d * p.rep + rr);
            if ((uint64_t)(uint32_t)pr.y >= ds.nblocks) {
                bad = true;
                continue;
            }
            char* dp = reinterpret_cast<char*>(ds.base + (int64_t)pr.y * ds.bstride + off);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t o = (u * 32 + lane) * 16;
                if (o < len) st_stream(dp + o, v[u]);
            }
        }
    }
    if (bad && lane == 0) atomicOr(p.err, kErrBadBlock);
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
cudaError_t launch_demand_scan(const int32_t* seq_lens, int32_t num_seqs, int32_t block_size, int32_t max_blocks,
                               int64_t avail_blocks, int32_t* off, int32_t* total, uint32_t* err,
                               cudaStream_t stream) {
    demand_scan_kernel<<<1, kScanThreads, 0, stream>>>(seq_lens, num_seqs, block_size, max_blocks, avail_blocks, off,
                                                       total, err);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_remap_tables(const int32_t* block_tables, int32_t num_seqs, int32_t max_blocks, int32_t base_block,
                                const int32_t* off, int32_t* dst_block_tables, int2* pairs, uint32_t* err,
                                cudaStream_t stream) {
    if (num_seqs == 0 || max_blocks == 0) return cudaSuccess;
    const int warps_per_cta = kRemapThreads / 32;
    int64_t blocks = ((int64_t)num_seqs + warps_per_cta - 1) / warps_per_cta;
    const int grid = (int)(blocks < 65536 ? blocks : 65536);  // the kernel strides over the rest
    remap_tables_kernel<<<grid, kRemapThreads, 0, stream>>>(block_tables, num_seqs, max_blocks, base_block, off,
                                                            dst_block_tables, pairs, err);
    count_launch();
    return cudaGetLastError();
}

template <int U>
static cudaError_t launch_regcopy(const MigrateParams& p, const LaunchCfg& cfg, cudaStream_t stream) {
    int per_sm = cfg.ctas_per_sm;
    if (per_sm <= 0) {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, migrate_regcopy_kernel<U>, kCopyThreads, 0);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) per_sm = 1;
    }
    migrate_regcopy_kernel<U><<<cfg.num_sms * per_sm, kCopyThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_migrate(const MigrateParams& p, const LaunchCfg& cfg, cudaStream_t stream) {
    switch (p.chunk_bytes) {
        case 1024: return launch_regcopy<2>(p, cfg, stream);
        case 2048: return launch_regcopy<4>(p, cfg, stream);
        case 4096: return launch_regcopy<8>(p, cfg, stream);
        case 8192: return launch_regcopy<16>(p, cfg, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace remp
