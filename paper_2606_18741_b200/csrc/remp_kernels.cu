// Device kernels of libremp for sm_100a: block-demand prefix scan, block-table remapper (as separate launches
// and fused into one cluster launch for small inputs), and the KV migration (gather/scatter copy) kernels.

#include <cooperative_groups.h>

#include <algorithm>
#include <utility>

#include "remp_internal.h"

namespace cg = cooperative_groups;

namespace remp {

// ---------------------------------------------------------------------------------------------
// K1: demand[s] = ceil(len[s] / block_size); off = exclusive prefix sum; total; capacity check.
// One CTA walks the sequences in tiles of kScanThreads with a running carry, so the result is the plain
// serial sum in sequence order and needs no inter-CTA communication.
// ---------------------------------------------------------------------------------------------
constexpr int kScanThreads = 1024;
constexpr int kMultiCtaScanFrom = 8192;  // more sequences than this: three-launch scan over all SMs

__global__ void __launch_bounds__(kScanThreads) demand_scan_kernel(const int32_t* __restrict__ seq_lens,
                                                                  int32_t num_seqs, int32_t block_size,
                                                                  int32_t max_blocks, int64_t avail_blocks,
                                                                  int32_t preempt, int32_t* __restrict__ off,
                                                                  int32_t* __restrict__ total,
                                                                  uint32_t* __restrict__ err) {
    __shared__ long long warp_sum[kScanThreads / 32];
    __shared__ long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    uint32_t bad = 0;
    long long fit = 0;  // preempt mode: largest inclusive prefix sum that still fits (prefix sums never decrease)
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
        if (s < num_seqs) {
            off[s] = before > 0x7fffffffLL ? 0x7fffffff : (int32_t)before;
            if (before + need <= avail_blocks) fit = before + need;
        }
        __syncthreads();
        if (tid == kScanThreads - 1) carry_s = carry + warp_sum[kScanThreads / 32 - 1];
        __syncthreads();
    }
    const long long sum = carry_s;
    if (sum > 0x7fffffffLL) bad |= kErrOverflow;
    // block-wide maximum of `fit`
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) fit = max(fit, __shfl_xor_sync(0xffffffffu, fit, d));
    __syncthreads();
    if (lane == 0) warp_sum[wid] = fit;
    __syncthreads();
    if (tid == 0) {
        for (int i = 1; i < kScanThreads / 32; ++i) fit = max(fit, warp_sum[i]);
        if (!preempt && sum > avail_blocks) bad |= kErrCapacity;
        off[num_seqs] = sum > 0x7fffffffLL ? 0x7fffffff : (int32_t)sum;
        // blocks that will be allocated: everything, or (capacity-constrained) the longest prefix that fits
        const long long kept = preempt ? fit : sum;
        *total = (bad & kErrOverflow) && !preempt ? 0 : (int32_t)min(kept, 0x7fffffffLL);
    }
    if (preempt) bad &= ~kErrOverflow;  // a prefix that fits the pools fits 32 bits; only it is allocated
    if (bad) atomicOr(err, bad);
}

// ---------------------------------------------------------------------------------------------
// K1 for many sequences: the same sums in three launches without any inter-CTA wait. (a) every CTA sums the
// demand of its tile of kScanThreads sequences; (b) one CTA scans the tile sums (running carry), checks
// capacity and writes the total; (c) every CTA scans its tile again on top of its tile offset and writes
// off[]. Integer sums are associative, so off[] and the total are bit-identical to the one-CTA scan.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ long long demand_of(const int32_t* seq_lens, int32_t s, int32_t num_seqs,
                                               int32_t block_size, int32_t max_blocks, uint32_t* bad) {
    if (s >= num_seqs) return 0;
    const int32_t len = seq_lens[s];
    if (len < 0) {
        *bad |= kErrBadLength;
        return 0;
    }
    const long long need = ((long long)len + block_size - 1) / block_size;
    if (need > max_blocks) {
        *bad |= kErrBadLength;
        return 0;
    }
    return need;
}

// Inclusive scan of v over the CTA (kScanThreads threads); warp_sum is shared scratch of kScanThreads/32 entries.
// Returns the inclusive value of this thread; *tile_total receives the sum over the CTA.
__device__ __forceinline__ long long block_inclusive_scan(long long v, long long* warp_sum, long long* tile_total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    long long incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const long long up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    __syncthreads();  // warp_sum may still be read by a previous call
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        long long w = warp_sum[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const long long up = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += up;
        }
        warp_sum[lane] = w;
    }
    __syncthreads();
    *tile_total = warp_sum[kScanThreads / 32 - 1];
    return incl + (wid ? warp_sum[wid - 1] : 0);
}

__global__ void __launch_bounds__(kScanThreads) demand_tile_sums_kernel(const int32_t* __restrict__ seq_lens,
                                                                       int32_t num_seqs, int32_t block_size,
                                                                       int32_t max_blocks,
                                                                       long long* __restrict__ tile_sum,
                                                                       uint32_t* __restrict__ err) {
    __shared__ long long warp_sum[kScanThreads / 32];
    uint32_t bad = 0;
    const int32_t s = blockIdx.x * kScanThreads + threadIdx.x;
    const long long need = demand_of(seq_lens, s, num_seqs, block_size, max_blocks, &bad);
    long long total;
    block_inclusive_scan(need, warp_sum, &total);
    if (threadIdx.x == 0) tile_sum[blockIdx.x] = total;
    if (bad) atomicOr(err, bad);
}

__global__ void __launch_bounds__(kScanThreads) demand_tile_scan_kernel(long long* __restrict__ tile_sum,
                                                                       int32_t num_tiles, int64_t avail_blocks,
                                                                       int32_t preempt, int32_t num_seqs,
                                                                       int32_t* __restrict__ off,
                                                                       int32_t* __restrict__ total,
                                                                       uint32_t* __restrict__ err) {
    __shared__ long long warp_sum[kScanThreads / 32];
    __shared__ long long carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int32_t base = 0; base < num_tiles; base += kScanThreads) {
        const int32_t t = base + threadIdx.x;
        const long long v = t < num_tiles ? tile_sum[t] : 0;
        long long tile_total;
        const long long incl = block_inclusive_scan(v, warp_sum, &tile_total);
        const long long carry = carry_s;
        if (t < num_tiles) tile_sum[t] = carry + incl - v;  // exclusive offset of tile t, in place
        __syncthreads();
        if (threadIdx.x == 0) carry_s = carry + tile_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const long long sum = carry_s;
        uint32_t bad = 0;
        if (sum > 0x7fffffffLL && !preempt) bad |= kErrOverflow;
        if (!preempt && sum > avail_blocks) bad |= kErrCapacity;
        off[num_seqs] = sum > 0x7fffffffLL ? 0x7fffffff : (int32_t)sum;
        // capacity-constrained mode: the apply kernel raises the total to the longest prefix that fits
        *total = preempt ? 0 : ((bad & kErrOverflow) ? 0 : (int32_t)sum);
        if (bad) atomicOr(err, bad);
    }
}

__global__ void __launch_bounds__(kScanThreads) demand_apply_kernel(const int32_t* __restrict__ seq_lens,
                                                                   int32_t num_seqs, int32_t block_size,
                                                                   int32_t max_blocks,
                                                                   const long long* __restrict__ tile_off,
                                                                   int64_t avail_blocks, int32_t preempt,
                                                                   int32_t* __restrict__ off,
                                                                   int32_t* __restrict__ total) {
    __shared__ long long warp_sum[kScanThreads / 32];
    uint32_t bad = 0;  // lengths were already reported by the first pass
    const int32_t s = blockIdx.x * kScanThreads + threadIdx.x;
    const long long need = demand_of(seq_lens, s, num_seqs, block_size, max_blocks, &bad);
    long long tile_total;
    const long long incl = block_inclusive_scan(need, warp_sum, &tile_total);
    const long long before = tile_off[blockIdx.x] + incl - need;
    if (s < num_seqs) {
        off[s] = before > 0x7fffffffLL ? 0x7fffffff : (int32_t)before;
        if (preempt && before + need <= avail_blocks) atomicMax(total, (int32_t)min(before + need, 0x7fffffffLL));
    }
}

// ---------------------------------------------------------------------------------------------
// K2: one warp per sequence. dst_bt[s][j] = base + off[s] + j for live entries, -1 for padding; the
// flat pair list pairs[off[s] + j] = (source block, destination block) drives the migration kernel.
// Writes nothing when the scan recorded a fatal condition (capacity, bad length, overflow).
// ---------------------------------------------------------------------------------------------
constexpr int kRemapThreads = 256;
constexpr int kRemapSegment = 256;  // table columns one warp handles

__global__ void __launch_bounds__(kRemapThreads) remap_tables_kernel(const int32_t* __restrict__ block_tables,
                                                                    int32_t num_seqs, int32_t max_blocks,
                                                                    int32_t base_block,
                                                                    const int32_t* __restrict__ off,
                                                                    int32_t* __restrict__ dst_block_tables,
                                                                    int4* __restrict__ pairs,
                                                                    uint32_t* __restrict__ err,
                                                                    const int32_t* __restrict__ seq_lens,
                                                                    int32_t block_size, int64_t keep_below,
                                                                    int32_t* __restrict__ preempted,
                                                                    uint32_t* __restrict__ num_preempted) {
    // keep_below < 0: every sequence is allocated. Otherwise (capacity-constrained): sequence s is kept iff the
    // blocks of sequences 0..s fit, off[s+1] <= keep_below; the others get an all -1 row and preempted[s] = 1.
    if (*reinterpret_cast<volatile uint32_t*>(err) & kErrFatalMask) return;
    // One warp per (sequence, segment of kRemapSegment table columns), so that a few very wide rows still
    // spread over the GPU.
    const int lane = threadIdx.x & 31;
    const int32_t warps_per_cta = kRemapThreads / 32;
    const int64_t nwarps = (int64_t)gridDim.x * warps_per_cta;
    const int64_t nseg = max_blocks > 0 ? (max_blocks + kRemapSegment - 1) / kRemapSegment : 1;
    const int64_t units = (int64_t)num_seqs * nseg;
    bool bad = false;
    for (int64_t u = (int64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5); u < units; u += nwarps) {
        const int64_t s = u / nseg;
        const int32_t col0 = (int32_t)(u - s * nseg) * kRemapSegment;
        int32_t o0 = 0, o1 = 0, len = 0;
        if (lane == 0) {
            o0 = off[s];
            o1 = off[s + 1];
            len = seq_lens[s];
        }
        o0 = __shfl_sync(0xffffffffu, o0, 0);
        o1 = __shfl_sync(0xffffffffu, o1, 0);
        len = __shfl_sync(0xffffffffu, len, 0);
        int32_t need = o1 - o0;
        if (keep_below >= 0) {
            const bool out_ = (int64_t)o1 > keep_below;
            if (out_) need = 0;
            if (lane == 0 && col0 == 0) {
                preempted[s] = out_ ? 1 : 0;
                if (out_) atomicAdd(num_preempted, 1u);
            }
        }
        const int32_t* row = block_tables + s * max_blocks;
        int32_t* out = dst_block_tables + s * max_blocks;
        const int32_t col1 = min(max_blocks, col0 + kRemapSegment);
        for (int32_t j = col0 + lane; j < col1; j += 32) {
            if (j < need) {
                int32_t sb = row[j];
                const int32_t db = base_block + o0 + j;
                if (sb < 0) {
                    bad = true;
                    sb = -1;
                }
                out[j] = db;
                pairs[o0 + j] = make_int4(sb, db, min(block_size, len - j * block_size), 0);  // tokens in use
            } else {
                out[j] = -1;
            }
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(err, kErrBadBlock);
}

// ---------------------------------------------------------------------------------------------
// K1 + K2 in one launch, for at most kFusedMaxSeqs sequences: a small switch is bound by launch gaps, not by
// work, so the whole allocation is one kernel and needs no memset before it. The grid is ONE thread-block
// cluster of 1..8 CTAs. Every CTA scans the (at most 1024) demands itself in shared memory - the sums are
// the serial ones, identical in every CTA - and then rewrites its share of the table rows. The only thing
// the CTAs have to tell each other is "I saw a negative source id": one flag per CTA, read by CTA 0 through
// distributed shared memory after a cluster barrier. CTA 0 then stores (not ORs) the error word, the total,
// the preempted count and the start state of the tile scheduler, so nothing has to be zeroed beforehand.
// ---------------------------------------------------------------------------------------------
constexpr int kFusedThreads = 1024;
static_assert(kFusedThreads == kScanThreads && kFusedMaxSeqs <= kFusedThreads, "one scan tile");

__global__ void __launch_bounds__(kFusedThreads) alloc_fused_kernel(
    const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ block_tables, int32_t num_seqs,
    int32_t max_blocks, int32_t block_size, int32_t base_block, int64_t avail_blocks, int32_t preempt,
    int32_t* __restrict__ off, int32_t* __restrict__ words, int32_t* __restrict__ dst_block_tables,
    int4* __restrict__ pairs, int32_t* __restrict__ preempted) {
    // the migration kernel behind this one in the stream may be set up while this one runs; it waits for this
    // kernel's completion before it reads anything written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t crank = cluster.block_rank(), csize = cluster.num_blocks();
    __shared__ long long warp_sum[kFusedThreads / 32];
    __shared__ int32_t s_off[kFusedMaxSeqs + 1];
    __shared__ int32_t s_len[kFusedMaxSeqs];
    __shared__ long long s_kept;
    __shared__ uint32_t s_flag;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

    // ---- demand and prefix sum (same values in every CTA) ----
    uint32_t bad = 0;
    const long long need = demand_of(seq_lens, tid, num_seqs, block_size, max_blocks, &bad);
    long long sum;
    const long long incl = block_inclusive_scan(need, warp_sum, &sum);
    const bool mine = tid < num_seqs;
    if (mine) {
        s_off[tid] = (int32_t)min(incl - need, 0x7fffffffLL);
        s_len[tid] = seq_lens[tid];
    }
    if (tid == 0) {
        s_off[num_seqs] = (int32_t)min(sum, 0x7fffffffLL);
        s_kept = 0;
    }
    uint32_t status = __syncthreads_or(bad != 0) ? kErrBadLength : 0;
    // capacity-constrained mode: prefix sums never decrease, so the kept sequences are the first n_keep ones
    const bool keep = !preempt || incl <= avail_blocks;
    const int n_keep = __syncthreads_count(mine && keep);
    if (preempt && mine && tid == n_keep - 1) s_kept = incl;
    __syncthreads();
    const long long kept = preempt ? s_kept : sum;
    if (!preempt) {
        if (sum > 0x7fffffffLL) status |= kErrOverflow;
        if (sum > avail_blocks) status |= kErrCapacity;
    }
    if (crank == 0) {  // results that do not depend on the table rows
        if (mine) {
            off[tid] = s_off[tid];
            if (preempt) preempted[tid] = keep ? 0 : 1;
        }
        if (tid == 0) {
            off[num_seqs] = s_off[num_seqs];
            words[kWordTotal] = (status & kErrOverflow) ? 0 : (int32_t)min(kept, 0x7fffffffLL);
            words[kWordPreempted] = preempt ? num_seqs - n_keep : 0;
            words[kWordSched] = 0;  // the 64-bit tile-scheduler word of the migration kernels
            words[kWordSched + 1] = 0;
            if (status & kErrFatalMask) words[kWordErr] = (int32_t)status;
        }
    }
    if (status & kErrFatalMask) return;  // every CTA of the cluster takes this branch or none does

    // ---- table rows: one warp per (sequence, segment of kRemapSegment columns), over the whole cluster ----
    const int64_t nseg = max_blocks > 0 ? (max_blocks + kRemapSegment - 1) / kRemapSegment : 1;
    const int64_t units = (int64_t)num_seqs * nseg;
    const int64_t nwarps = (int64_t)csize * (kFusedThreads / 32);
    bool badblk = false;
    for (int64_t u = (int64_t)crank * (kFusedThreads / 32) + wid; u < units; u += nwarps) {
        const int32_t s = (int32_t)(u / nseg);
        const int32_t col0 = (int32_t)(u - (int64_t)s * nseg) * kRemapSegment;
        const int32_t o0 = s_off[s], len = s_len[s];
        int32_t need_s = s_off[s + 1] - o0;
        if (preempt && s >= n_keep) need_s = 0;
        const int32_t* row = block_tables + (int64_t)s * max_blocks;
        int32_t* out = dst_block_tables + (int64_t)s * max_blocks;
        const int32_t col1 = min(max_blocks, col0 + kRemapSegment);
        for (int32_t j = col0 + lane; j < col1; j += 32) {
            if (j < need_s) {
                int32_t sb = row[j];
                const int32_t db = base_block + o0 + j;
                if (sb < 0) {
                    badblk = true;
                    sb = -1;
                }
                out[j] = db;
                pairs[o0 + j] = make_int4(sb, db, min(block_size, len - j * block_size), 0);  // tokens in use
            } else {
                out[j] = -1;
            }
        }
    }
    // ---- one flag per CTA to CTA 0, which stores the error word ----
    const int any = __syncthreads_or(badblk);
    if (csize == 1) {
        if (tid == 0) words[kWordErr] = (int32_t)(status | (any ? kErrBadBlock : 0u));
        return;
    }
    if (tid == 0) s_flag = any ? 1u : 0u;
    cluster.sync();
    if (crank == 0 && tid == 0) {
        uint32_t f = 0;
        for (uint32_t r = 0; r < csize; ++r) f |= *cluster.map_shared_rank(&s_flag, r);
        words[kWordErr] = (int32_t)(status | (f ? kErrBadBlock : 0u));
    }
    cluster.sync();  // the other CTAs' shared memory must outlive CTA 0's reads
}

// ---------------------------------------------------------------------------------------------
// K3 addressing. A work item names a destination plane g (stage, head-owner group, layer, K/V in the order
// the host laid the plane groups out) and a run `sub` of heads inside a block. locate() finds the source
// address of that run and what is needed to address each destination replica, from the small tables of
// MigrateParams (staged in shared memory, or in global memory when there are very many ranks).
// ---------------------------------------------------------------------------------------------
struct RunAddr {
    uint64_t base;    // address of the run in block 0
    int64_t bstride;  // bytes between consecutive blocks
    uint32_t nb;      // pool size in blocks (block ids are 32-bit, larger pools are clipped)
};
struct RunLoc {
    uint32_t rd0;  // index of the first destination replica's view
    uint32_t lloc, kv, hloc;
};

__device__ __forceinline__ const RankView* views_at(const uint8_t* tab, uint32_t off) {
    return reinterpret_cast<const RankView*>(tab + off);
}

__device__ __forceinline__ void locate(const MigrateParams& p, const uint8_t* tab, uint32_t plane, uint32_t sub,
                                       RunAddr* src, RunLoc* loc) {
    const PlaneGroup* pg = reinterpret_cast<const PlaneGroup*>(tab + p.off_group);
    uint32_t lo = 0, hi = p.n_pg;  // the last group that starts at or before `plane`
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (pg[mid].first_plane <= plane) lo = mid; else hi = mid;
    }
    const PlaneGroup G = pg[lo];
    const uint32_t rel = plane - G.first_plane, kv = rel & 1u, dl = rel >> 1;
    const uint32_t h = G.head0 + sub * p.run_heads;  // first head of the run
    const uint32_t qd = p.hl_dst_shift < 32 ? h >> p.hl_dst_shift : h / p.hl_dst;  // destination head-owner group
    loc->rd0 = G.rank0 + qd * p.rep;
    loc->lloc = G.lloc0 + dl;
    loc->kv = kv;
    loc->hloc = h - qd * p.hl_dst;
    // source: the lowest-numbered rank holding head h, in the stage that holds the layer
    const LayerSrc ls = reinterpret_cast<const LayerSrc*>(tab + p.off_layer)[G.layer0 + dl];
    const uint32_t qs = p.hl_src_shift < 32 ? h >> p.hl_src_shift : h / p.hl_src;  // hl_src is 1 when heads are replicated
    const RankView* v = views_at(tab, 0) + ls.rank0 + qs * p.rep_src;
    src->base = v->base + (int64_t)ls.lloc * v->s_layer + (int64_t)kv * v->s_kv + (int64_t)(h - qs * p.hl_src) * p.sh_src;
    src->bstride = v->s_block;
    src->nb = (uint32_t)min(v->nb, (uint64_t)0x80000000u);
}

// Replica rr of the run on the destination side. A replica whose rank lives on another GPU comes back with
// base == kViewElsewhere: the caller leaves it to that GPU.
__device__ __forceinline__ RunAddr dst_addr(const MigrateParams& p, const uint8_t* tab, const RunLoc& loc, uint32_t rr) {
    const RankView* v = views_at(tab, p.off_dst) + loc.rd0 + rr;
    RunAddr a;
    const uint64_t vb = v->base;
    a.base = vb == kViewElsewhere
                 ? kViewElsewhere
                 : vb + (int64_t)loc.lloc * v->s_layer + (int64_t)loc.kv * v->s_kv + (int64_t)loc.hloc * p.sh_dst;
    a.bstride = v->s_block;
    a.nb = (uint32_t)min(v->nb, (uint64_t)0x80000000u);
    return a;
}

// Start of every migration kernel. The kernel may have been launched while the allocation kernel before it in
// the stream was still running (programmatic dependent launch): everything up to here used only the kernel's
// own parameters; griddepcontrol.wait returns once the preceding kernel has completed and its writes are
// visible (at once when there is no such dependency). Then the live-block total and the error word, which sit
// side by side, come with one load. Returns false when a fatal condition was recorded (nothing may be copied).
__device__ __forceinline__ bool read_status(const MigrateParams& p, uint32_t* nb) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned long long w = *reinterpret_cast<const volatile unsigned long long*>(p.total);  // total | error word
    *nb = (uint32_t)w;
    return ((uint32_t)(w >> 32) & kErrFatalMask) == 0;
}

// The tables of this launch: copied from the kernel parameters into shared memory (a CTA-wide step, call it
// before any thread leaves), or read in place from global memory.
__device__ __forceinline__ const uint8_t* stage_tables(const MigrateParams& p, const TabPool& pool, uint4* s_tab) {
    if (p.gtab) return p.gtab;
    for (uint32_t i = threadIdx.x; i < (p.tab_bytes + 15) / 16; i += blockDim.x) s_tab[i] = pool.q[i];
    __syncthreads();
    return reinterpret_cast<const uint8_t*>(s_tab);
}

// Dynamic tile scheduler. The first tile of every CTA (or warp) is its own index; further tiles are drawn
// from the low half of the scheduler word. A CTA that has drawn its last tile adds one to the high half, and
// the last CTA to do so puts the word back to zero, so the next launch (ordered after this one) starts from
// zero without a memset. Both halves live in one word, so a thread's draws are ordered before its "finished"
// by the coherence order of that one address. No CTA waits for another.
__device__ __forceinline__ uint32_t draw_tile(const MigrateParams& p) { return (uint32_t)atomicAdd(p.sched, 1ull); }

template <bool SYNC>
__device__ __forceinline__ void finish_cta(const MigrateParams& p) {
    if (SYNC) __syncthreads();  // several threads of the CTA drew tiles
    if (threadIdx.x == 0) {
        const unsigned long long old = atomicAdd(p.sched, 1ull << 32);
        if ((uint32_t)(old >> 32) == gridDim.x - 1) atomicExch(p.sched, 0ull);
    }
}

// ---------------------------------------------------------------------------------------------
// K3, register-copy variant. Work item w = chunk `ch` of run `i` of live block `k` of destination
// plane `g`; w increases along destination addresses, and consecutive warps of the grid take
// consecutive items, so at any moment the whole GPU writes one narrow window of one destination plane
// and reads one source plane (TLB- and DRAM-page friendly). A warp moves one chunk per iteration with
// 16-byte streaming loads and stores, all loads of the chunk in flight before the first store.
// ---------------------------------------------------------------------------------------------
template <int VEC>
struct Vec;
template <>
struct Vec<16> {
    uint32_t r[4];
};
template <>
struct Vec<32> {
    uint32_t r[8];
};

template <int VEC>
__device__ __forceinline__ Vec<VEC> ld_stream(const void* p);
template <int VEC>
__device__ __forceinline__ void st_stream(void* p, const Vec<VEC>& v);

// 16-byte streaming accesses: read-only path, no L1 allocation; stores marked evict-first (cache-streaming).
template <>
__device__ __forceinline__ Vec<16> ld_stream<16>(const void* p) {
    Vec<16> v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3])
                 : "l"(p));
    return v;
}
template <>
__device__ __forceinline__ void st_stream<16>(void* p, const Vec<16>& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.r[0]), "r"(v.r[1]), "r"(v.r[2]), "r"(v.r[3])
                 : "memory");
}
// 32-byte accesses (sm_100): one instruction per 32 bytes, with an L2 evict-first priority.
template <>
__device__ __forceinline__ Vec<32> ld_stream<32>(const void* p) {
    Vec<32> v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]), "=r"(v.r[6]),
                   "=r"(v.r[7])
                 : "l"(p));
    return v;
}
template <>
__device__ __forceinline__ void st_stream<32>(void* p, const Vec<32>& v) {
    asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p),
                 "r"(v.r[0]), "r"(v.r[1]), "r"(v.r[2]), "r"(v.r[3]), "r"(v.r[4]), "r"(v.r[5]), "r"(v.r[6]), "r"(v.r[7])
                 : "memory");
}

// Valid-tokens-only mode, contiguous token rows: of a head slice only the first `used` bytes move. A 16-byte
// vector that starts at byte hb of its head slice is copied whole when it ends inside the used part, skipped
// when it starts outside, and when it straddles the end (token rows that are not a multiple of 16 bytes) it is
// loaded whole and only its first `used - hb` bytes are stored, one by one.
__device__ __forceinline__ uint32_t used_in_vec(uint32_t hb, uint32_t used) {
    return hb >= used ? 0u : min(16u, used - hb);
}
__device__ __forceinline__ void store_first_bytes(char* dp, const uint32_t (&r)[4], uint32_t n) {
    for (uint32_t b = 0; b < n; ++b) {
        const uint32_t word = b < 4 ? r[0] : b < 8 ? r[1] : b < 12 ? r[2] : r[3];
        dp[b] = (char)(word >> (8 * (b & 3)));
    }
}

// CTAs per SM a copy kernel is compiled for, by the 16-byte vectors a lane holds per item: a warp with few bytes
// in flight needs more warps beside it to keep the memory system busy, so small items trade registers for
// occupancy (1 vector: 6 CTAs = 48 warps, 2: 5, 4: 4, 8: 3, 16: 2).
__host__ __device__ constexpr int min_ctas_per_sm(int vectors) {
    return vectors <= 1 ? 6 : vectors <= 2 ? 5 : vectors <= 4 ? 4 : vectors <= 8 ? 3 : 2;
}

constexpr int kCopyThreads = 256;
constexpr int kCopyWarps = kCopyThreads / 32;  // the host computes MigrateParams.step_warps for 8 warps
static_assert(kCopyWarps == 8, "MigrateParams.step_warps is computed for 8 warps per CTA");

// Position of a work item: destination plane g, live block (or group of blocks) k, run i of the block, piece ch
// of the run. Work item w = ((g * n_k + k) * n_i + i) * n_ch + ch.
struct Cursor {
    uint32_t g, k, i, ch;
};

// A warp visits items t0 + warp, t0 + warp + stride, ... of a tile. The first one is decoded with divisions; the
// next is reached by adding the stride digit by digit in the mixed radix (n_k, n_i, n_ch): small items (1 KiB and
// less) cannot afford three integer divisions each. The digits of the stride come from the host (StepDigits).
struct Stepper {
    uint32_t n_k, n_i, n_ch;
    StepDigits d;
    __device__ __forceinline__ Cursor at(uint32_t w) const {
        const uint32_t per_block = n_i * n_ch, per_plane = n_k * per_block;
        Cursor c;
        c.g = w / per_plane;
        const uint32_t q = w - c.g * per_plane;
        c.k = per_block == 1 ? q : q / per_block;  // one run of one piece per block is the common case
        const uint32_t r = q - c.k * per_block;
        c.i = n_ch == 1 ? r : r / n_ch;
        c.ch = r - c.i * n_ch;
        return c;
    }
    __device__ __forceinline__ void advance(Cursor& c) const {
        c.ch += d.dch;
        c.i += d.di;
        if (c.ch >= n_ch) c.ch -= n_ch, ++c.i;
        c.k += d.dk;
        if (c.i >= n_i) c.i -= n_i, ++c.k;
        while (c.k >= n_k) c.k -= n_k, ++c.g;
    }
};

// The addresses of the run a warp worked on last, kept in shared memory (one record per warp): consecutive items
// of a warp usually stay in the same (plane, run) - always when the warp stride is a multiple of the runs per
// block - so the table walk of locate() is paid once per plane, not once per item, and costs no registers.
struct alignas(16) WarpRun {
    uint64_t src_base, dst_base;    // the run in block 0 of the source / of the first destination replica
    int64_t src_bstride, dst_bstride;
    uint32_t src_nb, dst_nb;
    RunLoc loc;                     // for the further replicas
};

// tag: the (plane, run) the record holds, as plane * n_sub + run; ~0u = nothing yet. Warp-uniform.
__device__ __forceinline__ void lookup(const MigrateParams& p, const uint8_t* tab, uint32_t g, uint32_t i, WarpRun* wr,
                                       uint32_t& tag, uint32_t lane) {
    const uint32_t key = g * p.n_sub + i;
    if (key == tag) return;
    RunAddr src;
    RunLoc loc;
    locate(p, tab, g, i, &src, &loc);
    const RunAddr d0 = dst_addr(p, tab, loc, 0);
    __syncwarp();  // nobody still reads the old record
    if (lane == 0) {
        wr->src_base = src.base, wr->src_bstride = src.bstride, wr->src_nb = src.nb;
        wr->dst_base = d0.base, wr->dst_bstride = d0.bstride, wr->dst_nb = d0.nb;
        wr->loc = loc;
    }
    __syncwarp();
    tag = key;
}

__device__ __forceinline__ RunAddr dst_of(const MigrateParams& p, const uint8_t* tab, const WarpRun* wr, uint32_t rr) {
    if (rr == 0) {
        RunAddr a;
        a.base = wr->dst_base, a.bstride = wr->dst_bstride, a.nb = wr->dst_nb;
        return a;
    }
    return dst_addr(p, tab, wr->loc, rr);
}

// One work item: gather the chunk into registers (all loads in flight before the first store), then store it
// to every destination replica. Returns false when a block id is out of range (the item is skipped).
// PARTIAL (valid-tokens-only mode): within every head slice of the run only the first `used` bytes move (used =
// tokens in use x bytes per token; a full block keeps everything).
//   1: a run is within one head slice and token rows are multiples of 16 bytes - the common case: the used part is
//      a prefix of the run in whole vectors, so the chunk is simply cut short (no per-vector work at all);
//   2: the general case (runs of several heads, narrow token rows): every vector is classified.
template <int U, int VEC, int PARTIAL>
__device__ __forceinline__ bool copy_item(const MigrateParams& p, const uint8_t* tab, const Cursor& c, WarpRun* wr,
                                          uint32_t& tag, uint32_t lane) {
    static_assert(!PARTIAL || VEC == 16, "the valid-tokens-only copy works on 16-byte vectors");
    struct {
        uint32_t off, len;
    } it;
    it.off = c.ch * p.chunk_bytes;
    it.len = min(p.chunk_bytes, p.run_bytes - it.off);
    const int4 pr = __ldg(p.pairs + c.k);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    if ((uint32_t)pr.x >= wr->src_nb) return false;  // also catches entries the remapper marked -1
    const uint32_t used = (uint32_t)pr.z * p.tok_bytes;
    const bool one_head = p.run_bytes <= p.head_bytes;
    if (PARTIAL && one_head && it.off >= used) return true;  // the whole chunk is slack
    if (PARTIAL == 1) it.len = min(it.len, used - it.off);   // the chunk ends where the tokens in use end
    auto part = [&](uint32_t o) -> uint32_t {  // bytes of the vector at chunk offset o that move
        if (PARTIAL != 2) return VEC;
        const uint32_t b = it.off + o;
        return used_in_vec(one_head ? b : b % p.head_bytes, used);
    };
    const char* sp = reinterpret_cast<const char*>(wr->src_base + (int64_t)pr.x * wr->src_bstride + it.off);
    Vec<VEC> v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t o = (u * 32 + lane) * VEC;
        if (o < it.len && part(o)) v[u] = ld_stream<VEC>(sp + o);
    }
    bool ok = true;
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
        if ((uint32_t)pr.y >= ds.nb) {
            ok = false;
            continue;
        }
        char* dp = reinterpret_cast<char*>(ds.base + (int64_t)pr.y * ds.bstride + it.off);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t o = (u * 32 + lane) * VEC;
            if (o < it.len) {
                const uint32_t n = part(o);
                if (n == VEC) {
                    st_stream<VEC>(dp + o, v[u]);
                } else if (PARTIAL == 2 && n) {
                    if constexpr (VEC == 16) store_first_bytes(dp + o, v[u].r, n);
                }
            }
        }
    }
    return ok;
}

// Contiguous runs of 16 .. 2048 bytes (a power of two): one work item is the same run of B = 2^bpi_shift
// CONSECUTIVE live blocks, B * run_bytes = up to 4 KiB, so that the per-item work (position, table lookup, pair
// records) is spent once per 4 KiB just as for long runs. Lane j holds the pair record of block j of the
// group; vector x of the item belongs to block x >> run_shift and fetches that block's ids with a shuffle.
template <int U>
__device__ __forceinline__ bool copy_blocks_item(const MigrateParams& p, const uint8_t* tab, const Cursor& c, WarpRun* wr,
                                                 uint32_t& tag, uint32_t nb, uint32_t lane) {
    const uint32_t k0 = c.k << p.bpi_shift;  // first block of group c.k; run c.i
    int4 mine = make_int4(-1, -1, 0, 0);
    if (lane < p.blocks_per_item && k0 + lane < nb) mine = __ldg(p.pairs + k0 + lane);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    const uint32_t in_run = (1u << p.run_shift) - 1;  // vectors per run - 1
    const uint32_t live = min(p.blocks_per_item, nb - k0) << p.run_shift;  // vectors of this item that exist
    const uint64_t sbase = wr->src_base;
    const int64_t sstride = wr->src_bstride;
    const uint32_t snb = wr->src_nb;
    Vec<16> v[U];
    bool fine = true;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t x = u * 32 + lane;
        const uint32_t sb = (uint32_t)__shfl_sync(0xffffffffu, mine.x, (x >> p.run_shift) & 31);
        if (x < live) {
            if (sb < snb)
                v[u] = ld_stream<16>(reinterpret_cast<const char*>(sbase + (int64_t)sb * sstride) + ((x & in_run) << 4));
            else
                fine = false;
        }
    }
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t x = u * 32 + lane;
            const uint32_t from = (x >> p.run_shift) & 31;
            const uint32_t sb = (uint32_t)__shfl_sync(0xffffffffu, mine.x, from);
            const uint32_t db = (uint32_t)__shfl_sync(0xffffffffu, mine.y, from);
            if (x < live && sb < snb) {
                if (db < ds.nb)
                    st_stream<16>(reinterpret_cast<char*>(ds.base + (int64_t)db * ds.bstride) + ((x & in_run) << 4), v[u]);
                else
                    fine = false;
            }
        }
    }
    return fine;
}

// DYNAMIC = false: tile t of a CTA is blockIdx + i * gridDim (static round-robin).
// DYNAMIC = true : CTAs draw tile numbers from a global counter, so faster SMs take more tiles and the
//                  whole GPU stays on one moving frontier until the last tile (the next tile number is
//                  fetched while the current tile is being copied).
//           = 2     : every warp draws its own tiles (no CTA barrier).
// PARTIAL: valid-tokens-only mode (0 off, 1 whole-vector prefix of a one-head run, 2 general; see copy_item).
// MULTI: short runs, an item is a run of several consecutive blocks (copy_blocks_item).
template <int U, int VEC, int DYNAMIC, int PARTIAL, bool MULTI = false>  // U vectors of VEC bytes per lane and item
__global__ void __launch_bounds__(kCopyThreads, min_ctas_per_sm(U * VEC / 16))
    migrate_regcopy_kernel(const __grid_constant__ MigrateParams p, const __grid_constant__ TabPool pool) {
    static_assert(!MULTI || (VEC == 16 && !PARTIAL), "multi-block items: 16-byte vectors, whole blocks");
    __shared__ uint4 s_tab[kTabBytes / 16];
    const uint8_t* tab = stage_tables(p, pool, s_tab);
    uint32_t nb;
    if (!read_status(p, &nb)) return;
    // MULTI: an item is (plane, group of blocks, run); else (plane, block, run, chunk of the run)
    const uint32_t n_k = MULTI ? (nb + p.blocks_per_item - 1) >> p.bpi_shift : nb;
    const uint32_t n_ch = MULTI ? 1u : p.nchunk;
    const uint32_t n_items = n_k * p.n_sub * n_ch * p.n_groups;  // < 2^32 - 2^22, checked on the host
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t tile = p.tile_items;  // consecutive items one CTA takes at a time
    const uint32_t n_tiles = n_items / tile + (n_items % tile ? 1u : 0u);
    bool bad = false;
    __shared__ WarpRun s_run[kCopyWarps];
    WarpRun* wr = s_run + warp;
    uint32_t tag = ~0u;
    const Stepper st{n_k, p.n_sub, n_ch, DYNAMIC == 2 ? p.step1 : p.step_warps};
    // the items a, a + stride, ... below t1 of tile t (32-bit arithmetic: t < n_tiles keeps t * tile below n_items)
    auto run_tile = [&](uint32_t t, uint32_t first, uint32_t stride) {
        const uint32_t t0 = t * tile, t1 = n_items - t0 < tile ? n_items : t0 + tile;
        if (first >= t1 - t0) return;
        Cursor c = st.at(t0 + first);
        for (uint32_t w = t0 + first; w < t1; w += stride) {
            if constexpr (MULTI)
                bad |= !copy_blocks_item<U>(p, tab, c, wr, tag, nb, lane);
            else
                bad |= !copy_item<U, VEC, PARTIAL>(p, tab, c, wr, tag, lane);
            st.advance(c);
        }
    };
    if (DYNAMIC == 2) {
        const uint32_t first_drawn = gridDim.x * kCopyWarps;  // tiles below this belong to the warps by index
        uint32_t nxt = blockIdx.x * kCopyWarps + warp;
        for (;;) {
            const uint32_t t = __shfl_sync(0xffffffffu, nxt, 0);
            if (t >= n_tiles) break;
            if (lane == 0) nxt = first_drawn + draw_tile(p);
            run_tile(t, 0, 1);
        }
    } else if (DYNAMIC == 1) {
        __shared__ uint32_t next_tile[2];
        if (threadIdx.x == 0) next_tile[0] = blockIdx.x;
        __syncthreads();
        for (uint32_t buf = 0;; buf ^= 1) {
            const uint32_t t = next_tile[buf];
            if (t >= n_tiles) break;
            if (threadIdx.x == 0) next_tile[buf ^ 1] = gridDim.x + draw_tile(p);
            run_tile(t, warp, kCopyWarps);
            __syncthreads();  // next_tile[buf ^ 1] is visible, next_tile[buf] may be overwritten
        }
    } else {
        for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x) run_tile(t, warp, kCopyWarps);
    }
    if (bad && lane == 0) atomicOr(p.err, kErrBadBlock);
    if (DYNAMIC) finish_cta<DYNAMIC == 2>(p);
}

// ---------------------------------------------------------------------------------------------
// K3, strided-row variant: the head and token strides of the two sides differ from the dense head-major
// block (token-major blocks [token][head][dim], padded heads ...), so a run is not one contiguous range
// but `rows` rows of row_bytes (the host folds every contiguous dimension into the row). A work item is 4 KiB of
// the run's rows taken back to back (256 vectors, whatever the row length: no lane idles because a row is not a
// power of two), or the whole run when it is shorter; a warp
// gathers the item's 16-byte vectors into registers (all loads first) and scatters them. Same frontier
// order and dynamic tile scheduler as the contiguous kernel.
// ---------------------------------------------------------------------------------------------
// Bytes of the 16-byte vector at (row i1/i2, column col) that move in valid-tokens-only mode (16 = all).
// PARTIAL 1: a row belongs to one token (token-major blocks, layout conversions), so a vector moves whole or not
// at all; PARTIAL 2: the tokens lie inside the row (strided heads), the last vector in use may move in part.
template <int PARTIAL>
__device__ __forceinline__ uint32_t row_vec_bytes(const MigrateParams& p, uint32_t vtok, uint32_t i1, uint32_t i2,
                                                  uint32_t col) {
    if (PARTIAL == 1) return (p.tok_mode == 1 ? i1 : i2) < vtok ? 16u : 0u;
    if (vtok >= p.block_size) return 16u;
    if (p.tok_mode == 0) return used_in_vec((col * 16) % p.head_bytes, vtok * p.tok_bytes);
    return (p.tok_mode == 1 ? i1 : i2) < vtok ? 16u : 0u;
}

// A destination offset (a multiple of 16 below 2^31) and the number of bytes of its vector that move (0..16) in
// one word: bit 31 = all 16 bytes, low four bits = 1..15 bytes (valid-tokens-only mode), neither = nothing.
__device__ __forceinline__ uint32_t pack_off(uint32_t doff, uint32_t nbytes) {
    return doff | (nbytes == 16 ? 0x80000000u : nbytes);
}
__device__ __forceinline__ uint32_t packed_off(uint32_t x) { return x & 0x7ffffff0u; }
__device__ __forceinline__ uint32_t packed_bytes(uint32_t x) { return (x >> 31) ? 16u : (x & 15u); }

// PARTIAL 2 = valid-tokens-only mode with tokens inside the rows; otherwise a vector moves whole or not at all.
template <int PARTIAL>
__device__ __forceinline__ void store_vec(char* dp, uint32_t packed, const Vec<16>& v) {
    if (PARTIAL == 2) {
        const uint32_t n = packed_bytes(packed);
        if (n == 16) st_stream<16>(dp + packed_off(packed), v);
        else if (n) store_first_bytes(dp + packed_off(packed), v.r, n);
    } else if (packed >> 31) {
        st_stream<16>(dp + packed_off(packed), v);
    }
}

// Where vector x of item q of a run lies inside a block, on both sides (a function of the run's row structure
// only, not of the block): source offset and pack_off(destination offset, 16 or 0).
__device__ __forceinline__ void row_vector(const MigrateParams& p, uint32_t q, uint32_t x, uint32_t* soff, uint32_t* doff) {
    const uint32_t vpr = p.row_bytes >> 4;  // 16-byte vectors per row
    const uint32_t gx = q * 256 + x;  // vector of the run: its rows back to back, 256 vectors per item
    const uint32_t row = p.vpr_shift < 32 ? gx >> p.vpr_shift : __umulhi(gx, p.vpr_magic), col = gx - row * vpr;
    const bool ok = row < p.rows;
    const uint32_t i1 = p.n2_shift < 32 ? row >> p.n2_shift : __umulhi(row, p.n2_magic), i2 = row - i1 * p.n2;
    *soff = i1 * p.s1 + i2 * p.s2 + col * 16;
    *doff = pack_off(i1 * p.d1 + i2 * p.d2 + col * 16, ok ? 16u : 0u);
}

// HOIST: the run fits one item (q is always 0) and whole blocks move, so the offsets of a lane's vectors are the
// same for every item: the kernel computed them once (pre_s, pre_d) and an item is just pair record, two base
// addresses, U loads and U stores - as cheap as a contiguous chunk.
template <int U>
__device__ __forceinline__ bool copy_rows_hoisted(const MigrateParams& p, const uint8_t* tab, const Cursor& c,
                                                  WarpRun* wr, uint32_t& tag, uint32_t lane, const uint32_t (&pre_s)[U],
                                                  const uint32_t (&pre_d)[U]) {
    const int4 pr = __ldg(p.pairs + c.k);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    if ((uint32_t)pr.x >= wr->src_nb) return false;
    const char* sp = reinterpret_cast<const char*>(wr->src_base + (int64_t)pr.x * wr->src_bstride);
    Vec<16> v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (pre_d[u] >> 31) v[u] = ld_stream<16>(sp + pre_s[u]);
    bool fine = true;
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
        if ((uint32_t)pr.y >= ds.nb) {
            fine = false;
            continue;
        }
        char* dp = reinterpret_cast<char*>(ds.base + (int64_t)pr.y * ds.bstride);
#pragma unroll
        for (int u = 0; u < U; ++u) store_vec<0>(dp, pre_d[u], v[u]);
    }
    return fine;
}

// AFFINE: rows of at most 512 bytes (a power of two) in one strided dimension, and an item is exactly U x 32
// vectors: vector u of a lane lies u * (32 / vectors per row) rows after vector 0, so its offsets are
// s0 + u * ds and d0 + u * dd - four registers instead of 2 U, and every vector of the item exists.
template <int U, int PARTIAL>
__device__ __forceinline__ bool copy_rows_affine(const MigrateParams& p, const uint8_t* tab, const Cursor& c,
                                                 WarpRun* wr, uint32_t& tag, uint32_t lane, uint32_t s0, uint32_t ds,
                                                 uint32_t d0, uint32_t dd) {
    static_assert(PARTIAL != 2, "affine rows: a row is one token's, vectors move whole");
    const int4 pr = __ldg(p.pairs + c.k);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    if ((uint32_t)pr.x >= wr->src_nb) return false;
    const char* sp = reinterpret_cast<const char*>(wr->src_base + (int64_t)pr.x * wr->src_bstride) + s0;
    // valid-tokens-only: row r is token r of the block; vector u of this lane lies in row r0 + u * rstep
    const uint32_t vtok = PARTIAL ? (uint32_t)pr.z : 0u;
    const uint32_t r0 = lane >> p.vpr_shift, rstep = 32u >> p.vpr_shift;
    Vec<16> v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (!PARTIAL || r0 + u * rstep < vtok) v[u] = ld_stream<16>(sp + u * ds);
    bool fine = true;
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds_ = dst_of(p, tab, wr, rr);
        if (ds_.base == kViewElsewhere) continue;
        if ((uint32_t)pr.y >= ds_.nb) {
            fine = false;
            continue;
        }
        char* dp = reinterpret_cast<char*>(ds_.base + (int64_t)pr.y * ds_.bstride) + d0;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (!PARTIAL || r0 + u * rstep < vtok) st_stream<16>(dp + u * dd, v[u]);
    }
    return fine;
}

// The same for items that span several consecutive blocks (MULTI): pre_s / pre_d are the offsets inside the
// vector's own block; the block ids come from the lanes' pair records by shuffle. Which block of the group a
// vector belongs to is a shift for power-of-two runs; otherwise (NP2) the kernel left it in the unused low bits of
// the offsets (bits 0-3 of pre_d, bit 0 of pre_s), so that no item pays a division for it.
template <int U, bool NP2>
__device__ __forceinline__ bool copy_rows_multi_hoisted(const MigrateParams& p, const uint8_t* tab, const Cursor& c,
                                                        WarpRun* wr, uint32_t& tag, uint32_t nb, uint32_t lane,
                                                        const uint32_t (&pre_s)[U], const uint32_t (&pre_d)[U]) {
    const uint32_t k0 = c.k * p.blocks_per_item;  // block group c.k, run c.i
    int4 mine = make_int4(-1, -1, 0, 0);
    if (lane < p.blocks_per_item && k0 + lane < nb) mine = __ldg(p.pairs + k0 + lane);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    const uint64_t sbase = wr->src_base;
    const int64_t sstride = wr->src_bstride;
    const uint32_t snb = wr->src_nb;
    const uint32_t nblk = min(p.blocks_per_item, nb - k0);  // blocks of this group that exist
    auto block_of = [&](int u) {
        if (!NP2) return (u * 32 + lane) >> p.run_shift;
        uint32_t lo = pre_d[u], hi = pre_s[u];
        asm volatile("" : "+r"(lo), "+r"(hi));  // decode per item: hoisted out of the item loop it costs 8 registers
        return (lo & 15u) | ((hi & 1u) << 4);
    };
    Vec<16> v[U];
    bool fine = true;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t b = block_of(u);
        const uint32_t sb = (uint32_t)__shfl_sync(0xffffffffu, mine.x, b & 31);
        if ((pre_d[u] >> 31) && b < nblk) {
            if (sb < snb)
                v[u] = ld_stream<16>(reinterpret_cast<const char*>(sbase + (int64_t)sb * sstride) + (NP2 ? pre_s[u] & ~15u : pre_s[u]));
            else
                fine = false;
        }
    }
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t b = block_of(u);
            const uint32_t sb = (uint32_t)__shfl_sync(0xffffffffu, mine.x, b & 31);
            const uint32_t db = (uint32_t)__shfl_sync(0xffffffffu, mine.y, b & 31);
            if ((pre_d[u] >> 31) && b < nblk && sb < snb) {
                if (db < ds.nb)
                    store_vec<0>(reinterpret_cast<char*>(ds.base + (int64_t)db * ds.bstride), pre_d[u], v[u]);
                else
                    fine = false;
            }
        }
    }
    return fine;
}

template <int U, int PARTIAL, bool MAGIC>
__device__ __forceinline__ bool copy_rows_item(const MigrateParams& p, const uint8_t* tab, const Cursor& c,
                                               WarpRun* wr, uint32_t& tag, uint32_t lane) {
    const uint32_t q = c.ch;  // item q of run c.i of block c.k
    const int4 pr = __ldg(p.pairs + c.k);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    if ((uint32_t)pr.x >= wr->src_nb) return false;
    const char* sp = reinterpret_cast<const char*>(wr->src_base + (int64_t)pr.x * wr->src_bstride);
    // valid-tokens-only: tokens at or beyond `vtok` of this block stay behind
    const uint32_t vtok = PARTIAL ? (uint32_t)pr.z : p.block_size;
    const uint32_t vpr = p.row_bytes >> 4;  // 16-byte vectors per row
    // divisions by vpr and n2 (uniform): shifts, or (MAGIC) multiplications by the host's reciprocals, divisor 1 aside
    auto div_vpr = [&](uint32_t x) { return !MAGIC ? x >> p.vpr_shift : p.vpr_shift == 0 ? x : __umulhi(x, p.vpr_magic); };
    auto div_n2 = [&](uint32_t x) { return !MAGIC ? x >> p.n2_shift : p.n2_shift == 0 ? x : __umulhi(x, p.n2_magic); };
    uint32_t doff[U];  // pack_off(destination offset, bytes that move)
    Vec<16> v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t x = u * 32 + lane;  // vector index inside the item
        const uint32_t gx = q * 256 + x;  // vector of the run: its rows back to back, 256 vectors per item
        const uint32_t row = div_vpr(gx), col = gx - row * vpr;
        const bool ok = row < p.rows;
        const uint32_t i1 = div_n2(row), i2 = row - i1 * p.n2;
        const uint32_t nbytes = !ok ? 0u : PARTIAL ? row_vec_bytes<PARTIAL>(p, vtok, i1, i2, col) : 16u;
        doff[u] = pack_off(i1 * p.d1 + i2 * p.d2 + col * 16, nbytes);
        if (nbytes) v[u] = ld_stream<16>(sp + (i1 * p.s1 + i2 * p.s2 + col * 16));
    }
    bool fine = true;
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
        if ((uint32_t)pr.y >= ds.nb) {
            fine = false;
            continue;
        }
        char* dp = reinterpret_cast<char*>(ds.base + (int64_t)pr.y * ds.bstride);
#pragma unroll
        for (int u = 0; u < U; ++u) store_vec<PARTIAL>(dp, doff[u], v[u]);
    }
    return fine;
}

// Runs shorter than 4 KiB: an item covers the same run of blocks_per_item consecutive live blocks, so that a
// warp still moves up to 4 KiB per iteration. Lane j holds the pair record of block j of the group; every
// vector fetches the record of its block with a shuffle.
template <int U, int PARTIAL, bool MAGIC>
__device__ __forceinline__ bool copy_rows_multi(const MigrateParams& p, const uint8_t* tab, const Cursor& c,
                                                WarpRun* wr, uint32_t& tag, uint32_t nb, uint32_t lane) {
    const uint32_t k0 = c.k * p.blocks_per_item;  // block group c.k, run c.i
    int4 mine = make_int4(-1, -1, 0, 0);
    if (lane < p.blocks_per_item && k0 + lane < nb) mine = __ldg(p.pairs + k0 + lane);
    lookup(p, tab, c.g, c.i, wr, tag, lane);
    const uint64_t sbase = wr->src_base;
    const int64_t sstride = wr->src_bstride;
    const uint32_t snb = wr->src_nb;
    const uint32_t vpr = p.row_bytes >> 4;
    const uint32_t vec_per_run = p.rows * vpr;
    const uint32_t live = min(p.blocks_per_item, nb - k0) * vec_per_run;  // vectors of this item that exist
    auto div_vpr = [&](uint32_t x) { return !MAGIC ? x >> p.vpr_shift : p.vpr_shift == 0 ? x : __umulhi(x, p.vpr_magic); };
    auto div_n2 = [&](uint32_t x) { return !MAGIC ? x >> p.n2_shift : p.n2_shift == 0 ? x : __umulhi(x, p.n2_magic); };
    auto div_run = [&](uint32_t x) { return !MAGIC ? x >> p.run_shift : p.run_shift == 0 ? x : __umulhi(x, p.run_magic); };
    uint32_t doff[U];  // pack_off(destination offset, bytes that move)
    Vec<16> v[U];
    bool fine = true;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t x = u * 32 + lane;  // vector index inside the item
        const uint32_t b = div_run(x), y = x - b * vec_per_run;
        const uint32_t row = div_vpr(y), col = y - row * vpr;
        const uint32_t sb = (uint32_t)__shfl_sync(0xffffffffu, mine.x, b & 31);
        const uint32_t vtok = PARTIAL ? (uint32_t)__shfl_sync(0xffffffffu, mine.z, b & 31) : p.block_size;
        bool ok = x < live;
        if (ok && sb >= snb) {
            fine = false;
            ok = false;
        }
        const uint32_t i1 = div_n2(row), i2 = row - i1 * p.n2;
        const uint32_t nbytes = !ok ? 0u : PARTIAL ? row_vec_bytes<PARTIAL>(p, vtok, i1, i2, col) : 16u;
        doff[u] = pack_off(i1 * p.d1 + i2 * p.d2 + col * 16, nbytes);
        if (nbytes)
            v[u] = ld_stream<16>(reinterpret_cast<const char*>(sbase + (int64_t)sb * sstride) +
                                 (i1 * p.s1 + i2 * p.s2 + col * 16));
    }
    for (uint32_t rr = 0; rr < p.rep; ++rr) {
        const RunAddr ds = dst_of(p, tab, wr, rr);
        if (ds.base == kViewElsewhere) continue;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t db = (uint32_t)__shfl_sync(0xffffffffu, mine.y, div_run(u * 32 + lane) & 31);
            if (!(doff[u] & 0x8000000fu)) continue;  // nothing of this vector moves
            if (db >= ds.nb) {
                fine = false;
                continue;
            }
            store_vec<PARTIAL>(reinterpret_cast<char*>(ds.base + (int64_t)db * ds.bstride), doff[u], v[u]);
        }
    }
    return fine;
}

// U: 16-byte vectors per lane per item (an item holds up to 512 * U bytes), chosen from the item size so that
// short runs do not pay for empty iterations.
// MULTI: items that span several blocks (runs of at most 2 KiB), compiled apart so that the common row
// kernel keeps its register budget. PARTIAL: valid-tokens-only mode.
// HOIST: whole blocks move and a run fits one item: per-lane vector offsets computed once per kernel (1; 3 for
// block groups of runs that are not a power of two), or, for short power-of-two rows in one strided dimension,
// reduced to an affine rule (2, copy_rows_affine). 0 and 5 are the general path, offsets computed per vector: 0 when
// every divisor (vectors per row, inner row count, vectors per run) is a power of two (shifts), 5 otherwise
// (multiplications by the reciprocals the host prepared).
template <int DYNAMIC, int U, bool MULTI, int PARTIAL, int HOIST>
__global__ void __launch_bounds__(kCopyThreads, MULTI && U >= 8 && (HOIST == 0 || HOIST == 5) ? 2 : min_ctas_per_sm(U)) migrate_rows_kernel(const __grid_constant__ MigrateParams p,
                                                                                  const __grid_constant__ TabPool pool) {
    __shared__ uint4 s_tab[kTabBytes / 16];
    const uint8_t* tab = stage_tables(p, pool, s_tab);
    uint32_t nb;
    if (!read_status(p, &nb)) return;
    constexpr bool multi = MULTI;
    const uint32_t per_block = p.n_sub * p.nchunk;
    const uint32_t per_plane = multi ? ((nb + p.blocks_per_item - 1) / p.blocks_per_item) * p.n_sub : nb * per_block;
    const uint32_t n_items = per_plane * p.n_groups;  // < 2^32 - 2^22, checked on the host
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t tile = p.tile_items;
    const uint32_t n_tiles = n_items / tile + (n_items % tile ? 1u : 0u);
    bool bad = false;
    __shared__ WarpRun s_run[kCopyWarps];
    WarpRun* wr = s_run + warp;
    uint32_t tag = ~0u;
    // MULTI: an item is (plane, group of blocks, run); else (plane, block, run, piece of the run)
    const Stepper st{multi ? (nb + p.blocks_per_item - 1) / p.blocks_per_item : nb, p.n_sub, multi ? 1u : p.nchunk,
                     p.step_warps};
    static_assert(!((HOIST == 1 || HOIST == 3) && PARTIAL) && !(HOIST == 2 && (MULTI || PARTIAL == 2)) &&
                      !(HOIST == 3 && !MULTI),
                  "hoisted offsets are for whole-block moves (affine ones also for whole token rows)");
    uint32_t pre_s[U], pre_d[U];  // HOIST: the offsets of this lane's vectors inside their block
    uint32_t s0 = 0, d0 = 0, ds = 0, dd = 0;  // HOIST == 2: vector u at s0 + u * ds / d0 + u * dd
    if (HOIST == 2) {
        uint32_t packed;
        row_vector(p, 0, lane, &s0, &packed);
        d0 = packed_off(packed);
        ds = (32u >> p.vpr_shift) * p.s1, dd = (32u >> p.vpr_shift) * p.d1;
    }
    if (HOIST == 1 || HOIST == 3) {
        const uint32_t vec_per_run = p.rows * (p.row_bytes >> 4);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t x = u * 32 + lane, b = 0;
            if (MULTI) {
                b = p.run_shift < 32 ? x >> p.run_shift : __umulhi(x, p.run_magic);
                x -= b * vec_per_run;
            }
            row_vector(p, 0, x, &pre_s[u], &pre_d[u]);
            if (MULTI && b >= p.blocks_per_item) pre_d[u] = 0;
            else if (MULTI && HOIST == 3) pre_d[u] |= b & 15u, pre_s[u] |= b >> 4;  // b <= 31, read back per item
        }
    }
    auto run_tile = [&](uint32_t t) {  // this warp's items of tile t: first + warp, + kCopyWarps, ...
        const uint32_t t0 = t * tile, t1 = n_items - t0 < tile ? n_items : t0 + tile;
        if (warp >= t1 - t0) return;
        Cursor c = st.at(t0 + warp);
        for (uint32_t w = t0 + warp; w < t1; w += kCopyWarps) {
            if constexpr (HOIST == 2)
                bad |= !copy_rows_affine<U, PARTIAL>(p, tab, c, wr, tag, lane, s0, ds, d0, dd);
            else if constexpr ((HOIST == 1 || HOIST == 3) && MULTI)
                bad |= !copy_rows_multi_hoisted<U, HOIST == 3>(p, tab, c, wr, tag, nb, lane, pre_s, pre_d);
            else if constexpr (HOIST == 1)
                bad |= !copy_rows_hoisted<U>(p, tab, c, wr, tag, lane, pre_s, pre_d);
            else if constexpr (MULTI)
                bad |= !copy_rows_multi<U, PARTIAL, HOIST == 5>(p, tab, c, wr, tag, nb, lane);
            else
                bad |= !copy_rows_item<U, PARTIAL, HOIST == 5>(p, tab, c, wr, tag, lane);
            st.advance(c);
        }
    };
    if (DYNAMIC) {
        __shared__ uint32_t next_tile[2];
        if (threadIdx.x == 0) next_tile[0] = blockIdx.x;
        __syncthreads();
        for (uint32_t buf = 0;; buf ^= 1) {
            const uint32_t t = next_tile[buf];
            if (t >= n_tiles) break;
            if (threadIdx.x == 0) next_tile[buf ^ 1] = gridDim.x + draw_tile(p);
            run_tile(t);
            __syncthreads();
        }
    } else {
        for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x) run_tile(t);
    }
    if (bad && lane == 0) atomicOr(p.err, kErrBadBlock);
    if (DYNAMIC) finish_cta<false>(p);
}

// ---------------------------------------------------------------------------------------------
// K3, bulk-copy variant: every participating thread owns one shared-memory stage and moves whole chunks
// with the bulk async-copy engine (cp.async.bulk, CTA-local): global -> its stage, completion on its
// own mbarrier, then stage -> every destination replica. No data passes through registers and one
// instruction moves a whole chunk. A CTA takes tiles of its stage count of consecutive items.
// Waits are bounded: a barrier that does not complete within p.wait_spins polls sets kErrWaitLimit; the
// thread then polls once more, up to the built-in limit, so that its load is no longer in flight when the CTA
// retires, copies nothing further and leaves the item's destination bytes as they were.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kWaitSpins = 1u << 20;  // try_wait itself suspends for a bounded time per call

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool bounded_wait(uint32_t bar_addr, uint32_t parity, uint32_t limit) {
    uint32_t done = 0;
    for (uint32_t spins = 0; !done && spins < limit; ++spins) {
        asm volatile(
            "{\n\t.reg .pred q;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, q;\n\t}"
            : "=r"(done)
            : "r"(bar_addr), "r"(parity)
            : "memory");
    }
    return done != 0;
}

// DYNAMIC: every warp draws tiles of LANES_PER_WARP consecutive items from the device counter (next tile
// prefetched) instead of striding by the grid; warps never wait for each other.
template <int LANES_PER_WARP, bool DYNAMIC>
__global__ void __launch_bounds__(1024) migrate_bulk_kernel(const __grid_constant__ MigrateParams p,
                                                            const __grid_constant__ TabPool pool, const uint32_t stages) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint4 s_tab[kTabBytes / 16];
    // layout: stages * chunk_bytes of data, then one 8-byte mbarrier per stage
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)stages * p.chunk_bytes);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool owner = lane < LANES_PER_WARP && warp * LANES_PER_WARP + lane < stages;
    const uint32_t slot = warp * LANES_PER_WARP + lane;
    if (owner) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + slot)));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint8_t* tab = stage_tables(p, pool, s_tab);
    __syncthreads();
    if (!owner) return;
    uint32_t nb;
    if (!read_status(p, &nb)) return;
    const uint32_t per_block = p.n_sub * p.nchunk;
    const uint32_t per_plane = nb * per_block;
    const uint64_t n_items = (uint64_t)per_plane * p.n_groups;
    const uint32_t stage_addr = smem_u32(smem + (size_t)slot * p.chunk_bytes);
    const uint32_t bar_addr = smem_u32(bars + slot);
    const uint32_t owners = __activemask();  // the stage-owning lanes of this warp
    const Stepper st{nb, p.n_sub, p.nchunk, p.step1};
    uint32_t parity = 0;
    uint32_t flags = 0;
    uint32_t nxt = 0;
    bool dead = false;  // a wait ran out: this lane stops issuing copies but keeps pace with its warp
    if (DYNAMIC && lane == 0) nxt = draw_tile(p);
    uint64_t w64 = (uint64_t)blockIdx.x * stages + slot;
    for (;;) {
        if (DYNAMIC) {
            const uint64_t t0 = (uint64_t)__shfl_sync(owners, nxt, 0) * LANES_PER_WARP;
            if (t0 >= n_items) break;
            if (lane == 0) nxt = draw_tile(p);
            w64 = t0 + lane;
            if (w64 >= n_items || dead) continue;  // ragged last tile, or given up: this lane sits the round out
        } else if (w64 >= n_items) {
            break;
        }
        const uint64_t w_now = w64;
        if (!DYNAMIC) w64 += (uint64_t)gridDim.x * stages;
        const Cursor c = st.at((uint32_t)w_now);
        struct {
            uint32_t k, off, len;
        } it;
        it.k = c.k;
        it.off = c.ch * p.chunk_bytes;
        it.len = min(p.chunk_bytes, p.run_bytes - it.off);
        const int4 pr = __ldg(p.pairs + it.k);
        RunAddr ss;
        RunLoc loc;
        locate(p, tab, c.g, c.i, &ss, &loc);
        if ((uint32_t)pr.x >= ss.nb) {
            flags |= kErrBadBlock;
            continue;
        }
        const uint64_t src = ss.base + (int64_t)pr.x * ss.bstride + it.off;
        // the stage is free once the previous stores have read it
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(it.len) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(stage_addr),
            "l"(src), "r"(it.len), "r"(bar_addr)
            : "memory");
        if (!bounded_wait(bar_addr, parity, p.wait_spins)) {
            // give up on this item; make sure the load has landed (or the built-in limit has passed) before this
            // thread can leave, and issue nothing more from this stage
            flags |= kErrWaitLimit;
            bounded_wait(bar_addr, parity, kWaitSpins);
            if (!DYNAMIC) break;
            dead = true;  // the other lanes of the warp still need this one at the tile hand-over
            continue;
        }
        parity ^= 1;
        for (uint32_t rr = 0; rr < p.rep; ++rr) {
            const RunAddr ds = dst_addr(p, tab, loc, rr);
            if (ds.base == kViewElsewhere) continue;
            if ((uint32_t)pr.y >= ds.nb) {
                flags |= kErrBadBlock;
                continue;
            }
            const uint64_t dst = ds.base + (int64_t)pr.y * ds.bstride + it.off;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(stage_addr),
                         "r"(it.len)
                         : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (flags) atomicOr(p.err, flags);
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
cudaError_t launch_demand_scan(const int32_t* seq_lens, int32_t num_seqs, int32_t block_size, int32_t max_blocks,
                               int64_t avail_blocks, int32_t* off, int32_t* total, uint32_t* err, cudaStream_t stream,
                               bool preempt, long long* tile_scratch) {
    if (tile_scratch && num_seqs > kMultiCtaScanFrom) {
        const int32_t tiles = (num_seqs + kScanThreads - 1) / kScanThreads;
        demand_tile_sums_kernel<<<tiles, kScanThreads, 0, stream>>>(seq_lens, num_seqs, block_size, max_blocks,
                                                                    tile_scratch, err);
        demand_tile_scan_kernel<<<1, kScanThreads, 0, stream>>>(tile_scratch, tiles, avail_blocks, preempt ? 1 : 0,
                                                                num_seqs, off, total, err);
        demand_apply_kernel<<<tiles, kScanThreads, 0, stream>>>(seq_lens, num_seqs, block_size, max_blocks, tile_scratch,
                                                                avail_blocks, preempt ? 1 : 0, off, total);
        count_launch(3);
        return cudaGetLastError();
    }
    demand_scan_kernel<<<1, kScanThreads, 0, stream>>>(seq_lens, num_seqs, block_size, max_blocks, avail_blocks,
                                                       preempt ? 1 : 0, off, total, err);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_remap_tables(const int32_t* block_tables, int32_t num_seqs, int32_t max_blocks, int32_t base_block,
                                const int32_t* off, int32_t* dst_block_tables, int4* pairs, uint32_t* err,
                                cudaStream_t stream, const int32_t* seq_lens, int32_t block_size, int64_t keep_below,
                                int32_t* preempted, uint32_t* num_preempted) {
    if (num_seqs == 0 || (max_blocks == 0 && keep_below < 0)) return cudaSuccess;
    const int warps_per_cta = kRemapThreads / 32;
    const int64_t nseg = max_blocks > 0 ? (max_blocks + kRemapSegment - 1) / kRemapSegment : 1;
    int64_t blocks = ((int64_t)num_seqs * nseg + warps_per_cta - 1) / warps_per_cta;
    const int grid = (int)(blocks < 65536 ? blocks : 65536);  // the kernel strides over the rest
    remap_tables_kernel<<<grid, kRemapThreads, 0, stream>>>(block_tables, num_seqs, max_blocks, base_block, off,
                                                            dst_block_tables, pairs, err, seq_lens, block_size,
                                                            keep_below, preempted, num_preempted);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_alloc_fused(const int32_t* seq_lens, const int32_t* block_tables, int32_t num_seqs,
                               int32_t max_blocks, int32_t block_size, int32_t base_block, int64_t avail_blocks,
                               bool preempt, int32_t* off, int32_t* words, int32_t* dst_block_tables, int4* pairs,
                               int32_t* preempted, cudaStream_t stream) {
    const int64_t nseg = max_blocks > 0 ? (max_blocks + kRemapSegment - 1) / kRemapSegment : 1;
    const int64_t units = (int64_t)num_seqs * nseg;
    if (num_seqs > kFusedMaxSeqs || (int64_t)num_seqs * max_blocks > kFusedMaxEntries) return cudaErrorNotSupported;
    // one cluster: a CTA per 64 (sequence, segment) units, at most the portable cluster size
    unsigned csize = 1;
    while (csize < 8 && (int64_t)csize * 64 < units) csize <<= 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(csize, 1, 1);
    cfg.blockDim = dim3(kFusedThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, alloc_fused_kernel, seq_lens, block_tables, num_seqs, max_blocks, block_size,
                                       base_block, avail_blocks, (int32_t)(preempt ? 1 : 0), off, words,
                                       dst_block_tables, pairs, preempted);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

// Launch a migration kernel so that it may be set up while the kernel before it in the stream (the allocation
// kernel of the same switch) is still running; the kernel itself waits for that kernel before it reads its
// results (read_status).
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int threads, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    if (e != cudaSuccess) return e;
    count_launch();
    return cudaGetLastError();
}

template <int U, int VEC, int DYNAMIC, int PARTIAL, bool MULTI = false>
static cudaError_t launch_regcopy_impl2(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg,
                                        cudaStream_t stream) {
    int per_sm = cfg.ctas_per_sm;
    if (per_sm <= 0) {
        static int cached = 0;  // a property of the kernel image, the same on every device of one kind
        if (!cached) {
            cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                &cached, migrate_regcopy_kernel<U, VEC, DYNAMIC, PARTIAL, MULTI>, kCopyThreads, 0);
            if (e != cudaSuccess) return e;
            if (cached < 1) cached = 1;
        }
        per_sm = cached;
    }
    const int64_t ctas_max = DYNAMIC == 2 ? (cfg.max_tiles + kCopyWarps - 1) / kCopyWarps : cfg.max_tiles;
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)cfg.num_sms * per_sm, ctas_max));
    return launch_dependent(migrate_regcopy_kernel<U, VEC, DYNAMIC, PARTIAL, MULTI>, grid, kCopyThreads, stream, p, tab);
}

template <int U, int VEC, int DYNAMIC>
static cudaError_t launch_regcopy_impl(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg,
                                       cudaStream_t stream) {
    if constexpr (VEC == 16) {
        // the used part of a block is a whole-vector prefix of every run: cut chunks short; else classify vectors
        if (p.valid_only && p.run_bytes <= p.head_bytes && p.tok_bytes % 16 == 0)
            return launch_regcopy_impl2<U, VEC, DYNAMIC, 1>(p, tab, cfg, stream);
        if (p.valid_only) return launch_regcopy_impl2<U, VEC, DYNAMIC, 2>(p, tab, cfg, stream);
    }
    return launch_regcopy_impl2<U, VEC, DYNAMIC, 0>(p, tab, cfg, stream);
}

// short contiguous runs: items of several consecutive blocks, U = vectors per lane (item bytes / 512)
template <int U>
static cudaError_t launch_blocks(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    if (cfg.dynamic == 2) return launch_regcopy_impl2<U, 16, 2, 0, true>(p, tab, cfg, stream);
    if (cfg.dynamic == 1) return launch_regcopy_impl2<U, 16, 1, 0, true>(p, tab, cfg, stream);
    return launch_regcopy_impl2<U, 16, 0, 0, true>(p, tab, cfg, stream);
}

template <int U, int VEC>
static cudaError_t launch_regcopy(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    if (cfg.dynamic == 2) return launch_regcopy_impl<U, VEC, 2>(p, tab, cfg, stream);
    if (cfg.dynamic == 1) return launch_regcopy_impl<U, VEC, 1>(p, tab, cfg, stream);
    return launch_regcopy_impl<U, VEC, 0>(p, tab, cfg, stream);
}

// Shared memory one CTA of the bulk-copy kernel may use for its stages when per_sm CTAs share an SM.
static size_t bulk_stage_budget(int per_sm) {
    return (size_t)(227 * 1024) / per_sm - (kTabBytes + 1024);  // the staged tables and the system's reserve
}

template <int LPW, bool DYNAMIC>
static cudaError_t launch_bulk_impl(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg,
                                    cudaStream_t stream) {
    // as many stages as fit the shared memory of one CTA per SM (or of ctas_per_sm CTAs)
    const int per_sm = cfg.ctas_per_sm > 0 ? cfg.ctas_per_sm : 1;
    const size_t budget = bulk_stage_budget(per_sm);
    uint32_t stages = (uint32_t)(budget / (p.chunk_bytes + 8));
    if (stages > 1024 / 32 * LPW) stages = 1024 / 32 * LPW;
    stages -= stages % LPW;  // every warp owns exactly LPW stages (a dynamic tile is LPW items)
    if (stages == 0) return cudaErrorInvalidValue;
    const uint32_t warps = (stages + LPW - 1) / LPW;
    const size_t smem = (size_t)stages * (p.chunk_bytes + 8);
    cudaError_t e =
        cudaFuncSetAttribute(migrate_bulk_kernel<LPW, DYNAMIC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    migrate_bulk_kernel<LPW, DYNAMIC><<<cfg.num_sms * per_sm, warps * 32, smem, stream>>>(p, tab, stages);
    count_launch();
    e = cudaGetLastError();
    // this kernel's warps draw tiles but do not put the scheduler word back: leave it at zero for the next launch
    if (e == cudaSuccess && DYNAMIC) e = cudaMemsetAsync(p.sched, 0, sizeof(unsigned long long), stream);
    return e;
}

template <int LPW>
static cudaError_t launch_bulk(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    return cfg.dynamic ? launch_bulk_impl<LPW, true>(p, tab, cfg, stream) : launch_bulk_impl<LPW, false>(p, tab, cfg, stream);
}

template <int DYNAMIC, int U, bool MULTI, int PARTIAL, int HOIST>
static cudaError_t launch_rows_impl(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    int per_sm = cfg.ctas_per_sm;
    if (per_sm <= 0) {
        static int cached = 0;
        if (!cached) {
            cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                &cached, migrate_rows_kernel<DYNAMIC, U, MULTI, PARTIAL, HOIST>, kCopyThreads, 0);
            if (e != cudaSuccess) return e;
            if (cached < 1) cached = 1;
        }
        per_sm = cached;
    }
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)cfg.num_sms * per_sm, cfg.max_tiles));
    return launch_dependent(migrate_rows_kernel<DYNAMIC, U, MULTI, PARTIAL, HOIST>, grid, kCopyThreads, stream, p, tab);
}

// The general path of the row kernel: divisions as shifts, or as multiplications when a divisor is not a power of two.
template <int DYNAMIC, int U, bool MULTI, int PARTIAL>
static cudaError_t launch_rows_general(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    const bool shifts = p.vpr_shift < 32 && p.n2_shift < 32 && (!MULTI || p.run_shift < 32);
    return shifts ? launch_rows_impl<DYNAMIC, U, MULTI, PARTIAL, 0>(p, tab, cfg, stream)
                  : launch_rows_impl<DYNAMIC, U, MULTI, PARTIAL, 5>(p, tab, cfg, stream);
}

template <int DYNAMIC, int U, bool MULTI>
static cudaError_t launch_rows_m(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    // short power-of-two rows in one strided dimension that fill a one-block item exactly: affine offsets
    // (one-block items hold more than 1 KiB; shorter runs move in block groups)
    const uint32_t vpr = p.row_bytes >> 4;
    const bool affine = !MULTI && U >= 4 && p.nchunk == 1 && p.n2 == 1 && p.vpr_shift < 32 && vpr <= 32 &&
                        p.rows * vpr == (uint32_t)U * 32;
    if (p.valid_only) {
        // tokens are whole rows (token-major blocks, layout conversions): vectors move whole or not at all
        if (p.tok_mode != 0) {
            if constexpr (!MULTI && U >= 4) {
                if (affine && p.tok_mode == 1) return launch_rows_impl<DYNAMIC, U, false, 1, 2>(p, tab, cfg, stream);
            }
            return launch_rows_general<DYNAMIC, U, MULTI, 1>(p, tab, cfg, stream);
        }
        return launch_rows_general<DYNAMIC, U, MULTI, 2>(p, tab, cfg, stream);
    }
    if constexpr (!MULTI && U >= 4) {
        if (affine) return launch_rows_impl<DYNAMIC, U, false, 0, 2>(p, tab, cfg, stream);
    }
    // whole blocks, and the run is one item: per-lane offsets are computed once per kernel
    if constexpr (MULTI) {
        if (p.run_shift >= 32) return launch_rows_impl<DYNAMIC, U, true, 0, 3>(p, tab, cfg, stream);
    }
    if (MULTI || p.nchunk == 1) return launch_rows_impl<DYNAMIC, U, MULTI, 0, 1>(p, tab, cfg, stream);
    return launch_rows_general<DYNAMIC, U, MULTI, 0>(p, tab, cfg, stream);
}

template <int DYNAMIC, int U>
static cudaError_t launch_rows_u(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    return p.blocks_per_item > 1 ? launch_rows_m<DYNAMIC, U, true>(p, tab, cfg, stream)
                                 : launch_rows_m<DYNAMIC, U, false>(p, tab, cfg, stream);
}

template <int DYNAMIC>
static cudaError_t launch_rows(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    // bytes one item holds: whole rows up to 4 KiB, or a 4 KiB piece of a long row; times the blocks of a group
    const uint32_t item_bytes = min(4096u, p.rows * p.row_bytes * max(1u, p.blocks_per_item));
    if (item_bytes <= 512) return launch_rows_u<DYNAMIC, 1>(p, tab, cfg, stream);
    if (item_bytes <= 1024) return launch_rows_u<DYNAMIC, 2>(p, tab, cfg, stream);
    if (item_bytes <= 2048) return launch_rows_u<DYNAMIC, 4>(p, tab, cfg, stream);
    return launch_rows_u<DYNAMIC, 8>(p, tab, cfg, stream);
}

bool regcopy_chunk_supported(int64_t chunk_bytes, int vec_bytes) {
    if (chunk_bytes != 512 && chunk_bytes != 1024 && chunk_bytes != 2048 && chunk_bytes != 4096 && chunk_bytes != 8192)
        return false;
    return vec_bytes != 32 || chunk_bytes >= 1024;
}

cudaError_t launch_migrate(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream) {
    if (cfg.kernel == 3) return cfg.dynamic ? launch_rows<1>(p, tab, cfg, stream) : launch_rows<0>(p, tab, cfg, stream);
    if (cfg.kernel == 2) {
        if (p.chunk_bytes % 16 != 0) return cudaErrorInvalidValue;
        // stages that fit one CTA bound the lanes per warp
        const int per_sm = cfg.ctas_per_sm > 0 ? cfg.ctas_per_sm : 1;
        const size_t budget = bulk_stage_budget(per_sm);
        int lpw = cfg.lanes_per_warp;
        while (lpw > 1 && (size_t)lpw * (p.chunk_bytes + 8) > budget) lpw >>= 1;
        switch (lpw) {
            case 1: return launch_bulk<1>(p, tab, cfg, stream);
            case 2: return launch_bulk<2>(p, tab, cfg, stream);
            case 4: return launch_bulk<4>(p, tab, cfg, stream);
            case 8: return launch_bulk<8>(p, tab, cfg, stream);
            case 16: return launch_bulk<16>(p, tab, cfg, stream);
            case 32: return launch_bulk<32>(p, tab, cfg, stream);
            default: return cudaErrorInvalidValue;
        }
    }
    if (cfg.kernel == 4) {  // multi-block items of short contiguous runs; chunk_bytes = bytes of one item
        switch (p.chunk_bytes) {
            case 512: return launch_blocks<1>(p, tab, cfg, stream);
            case 1024: return launch_blocks<2>(p, tab, cfg, stream);
            case 2048: return launch_blocks<4>(p, tab, cfg, stream);
            case 4096: return launch_blocks<8>(p, tab, cfg, stream);
            default: return cudaErrorInvalidValue;
        }
    }
    if (cfg.vec_bytes == 32) {
        switch (p.chunk_bytes) {
            case 1024: return launch_regcopy<1, 32>(p, tab, cfg, stream);
            case 2048: return launch_regcopy<2, 32>(p, tab, cfg, stream);
            case 4096: return launch_regcopy<4, 32>(p, tab, cfg, stream);
            case 8192: return launch_regcopy<8, 32>(p, tab, cfg, stream);
            default: return cudaErrorInvalidValue;
        }
    }
    switch (p.chunk_bytes) {
        case 512: return launch_regcopy<1, 16>(p, tab, cfg, stream);
        case 1024: return launch_regcopy<2, 16>(p, tab, cfg, stream);
        case 2048: return launch_regcopy<4, 16>(p, tab, cfg, stream);
        case 4096: return launch_regcopy<8, 16>(p, tab, cfg, stream);
        case 8192: return launch_regcopy<16, 16>(p, tab, cfg, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace remp
