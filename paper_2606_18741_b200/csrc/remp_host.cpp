// Host side of libremp: topology maps, the Algorithm-1 planner, and the C-ABI entry points.
// Device work is in remp_kernels.cu; this file only validates, plans, and enqueues.

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <numeric>

#include "remp_internal.h"

namespace remp {

static thread_local std::string g_last_error;
static std::atomic<int64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static remp_status fail(remp_status st, const std::string& msg) {
    g_last_error = msg;
    return st;
}

remp_status report_error(remp_status st, const char* msg) { return fail(st, msg); }

static remp_status cuda_fail(cudaError_t e, const char* what) {
    return fail(REMP_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define REMP_CUDA(call)                                     \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

// ---------------------------------------------------------------------------------------------
// Topology maps (section 3.4.1). Layers: contiguous ascending stages. Heads: even contiguous split,
// or one head per rank with rep consecutive ranks per head when TP exceeds the head count.
// ---------------------------------------------------------------------------------------------
remp_status build_topo_map(const remp_topo& t, const remp_model_shape& m, TopoMap* out, std::string* why) {
    const int L = m.num_layers, H = m.num_kv_heads;
    if (t.tp < 1 || t.pp < 1) {
        *why = "TP and PP must be >= 1";
        return REMP_ERR_INVALID_TOPOLOGY;
    }
    if (t.pp > L) {
        *why = "PP exceeds the number of layers";
        return REMP_ERR_INVALID_TOPOLOGY;
    }
    const bool split = t.tp <= H;
    if (split ? (H % t.tp != 0) : (t.tp % H != 0)) {
        *why = "TP must divide the KV-head count, or be a multiple of it";
        return REMP_ERR_INVALID_TOPOLOGY;
    }
    TopoMap T;
    T.tp = t.tp;
    T.pp = t.pp;
    T.heads_per_rank = split ? H / t.tp : 1;
    T.rep = split ? 1 : t.tp / H;
    T.layer_start.assign(t.pp + 1, 0);
    if (t.pp_layer_start) {
        for (int p = 0; p <= t.pp; ++p) T.layer_start[p] = t.pp_layer_start[p];
        bool ok = T.layer_start[0] == 0 && T.layer_start[t.pp] == L;
        for (int p = 0; p < t.pp && ok; ++p) ok = T.layer_start[p + 1] > T.layer_start[p];
        if (!ok) {
            *why = "pp_layer_start must rise strictly from 0 to num_layers";
            return REMP_ERR_INVALID_TOPOLOGY;
        }
    } else {
        const int q = L / t.pp, r = L % t.pp;
        for (int p = 0; p < t.pp; ++p) T.layer_start[p + 1] = T.layer_start[p] + q + (p < r ? 1 : 0);
    }
    T.stage_of_layer.resize(L);
    for (int p = 0; p < t.pp; ++p)
        for (int l = T.layer_start[p]; l < T.layer_start[p + 1]; ++l) T.stage_of_layer[l] = p;
    T.head_lo.resize(t.tp);
    T.first_owner.assign(H, -1);
    for (int r = t.tp - 1; r >= 0; --r) {  // descending, so the lowest owner is written last
        T.head_lo[r] = split ? r * T.heads_per_rank : r / T.rep;
        for (int h = T.head_lo[r]; h < T.head_lo[r] + T.heads_per_rank; ++h) T.first_owner[h] = r;
    }
    *out = std::move(T);
    return REMP_OK;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1: for every layer and destination TP rank, walk its head range and cut it at the
// boundaries of the source ranks' ranges; each piece is one item. A replicated source head yields one
// item only (from its lowest owner), so every destination slice has exactly one writer.
// ---------------------------------------------------------------------------------------------
static void build_items(const TopoMap& S, const TopoMap& D, int L, std::vector<Item>* items) {
    items->clear();
    for (int l = 0; l < L; ++l) {
        const int old_pp = S.stage_of_layer[l], new_pp = D.stage_of_layer[l];
        for (int ntp = 0; ntp < D.tp; ++ntp) {
            const int t_hi = D.head_lo[ntp] + D.heads_per_rank;
            int h = D.head_lo[ntp];
            while (h < t_hi) {
                const int otp = S.first_owner[h];
                const int hi = std::min(t_hi, S.head_lo[otp] + S.heads_per_rank);
                items->push_back(Item{S.rank(old_pp, otp), D.rank(new_pp, ntp), l, h, hi});
                h = hi;
            }
        }
    }
}

static int64_t dense_layer_bytes(const TopoMap& T, const remp_model_shape& m, int64_t nb) {
    return 2 * nb * T.heads_per_rank * (int64_t)m.block_size * m.head_dim * m.elem_bytes;
}

static remp_status check_shape(const remp_model_shape& m) {
    if (m.num_layers < 1 || m.num_kv_heads < 1 || m.head_dim < 1 || m.block_size < 1)
        return fail(REMP_ERR_SHAPE, "model dimensions must be positive");
    if (m.elem_bytes != 1 && m.elem_bytes != 2 && m.elem_bytes != 4)
        return fail(REMP_ERR_SHAPE, "elem_bytes must be 1, 2 or 4");
    const int64_t hs = (int64_t)m.block_size * m.head_dim * m.elem_bytes;
    if (hs % 16 != 0) return fail(REMP_ERR_SHAPE, "block_size*head_dim*elem_bytes must be a multiple of 16");
    if (hs * m.num_kv_heads > (int64_t)1 << 30) return fail(REMP_ERR_SHAPE, "a block of one layer exceeds 1 GiB");
    return REMP_OK;
}

}  // namespace remp

using namespace remp;

// Library-owned memory pools, one per device, created on first use (see device_pool).
static std::mutex g_pool_mu;
static cudaMemPool_t g_pools[64] = {};

// =============================================================================================
// C ABI
// =============================================================================================

extern "C" const char* remp_last_error(void) { return g_last_error.c_str(); }

extern "C" remp_status remp_release_cached_memory(void) {
    std::lock_guard<std::mutex> lock(g_pool_mu);
    for (cudaMemPool_t pool : g_pools)
        if (pool) REMP_CUDA(cudaMemPoolTrimTo(pool, 0));
    return REMP_OK;
}

extern "C" int64_t remp_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" int64_t remp_shard_bytes(const remp_topo* topo, const remp_model_shape* shape, int32_t rank,
                                    int64_t num_blocks) {
    if (!topo || !shape || num_blocks < 0) return fail(REMP_ERR_INVALID_ARG, "null argument or negative block count");
    if (remp_status st = check_shape(*shape)) return st;
    TopoMap T;
    std::string why;
    if (remp_status st = build_topo_map(*topo, *shape, &T, &why)) return fail(st, why);
    if (rank < 0 || rank >= T.num_ranks()) return fail(REMP_ERR_INVALID_ARG, "rank out of range");
    return T.stage_layers(rank / T.tp) * dense_layer_bytes(T, *shape, num_blocks);
}

static void release_scratch(remp_plan* P);

extern "C" void remp_plan_destroy(remp_plan* plan) {
    if (!plan) return;
    release_scratch(plan);
    delete plan;
}

extern "C" remp_status remp_plan_create(const remp_topo* src, const remp_topo* dst, const remp_model_shape* shape,
                                        const remp_block_tables* tables, remp_plan** out) {
    if (!src || !dst || !shape || !tables || !out) return fail(REMP_ERR_INVALID_ARG, "null argument");
    *out = nullptr;
    if (remp_status st = check_shape(*shape)) return st;
    if (tables->num_seqs < 0 || tables->max_blocks_per_seq < 0)
        return fail(REMP_ERR_INVALID_ARG, "negative table dimensions");
    if (tables->num_seqs > 0 && (!tables->seq_lens || (tables->max_blocks_per_seq > 0 && !tables->block_tables)))
        return fail(REMP_ERR_INVALID_ARG, "null seq_lens or block_tables");

    remp_plan* P = new (std::nothrow) remp_plan_s();
    if (!P) return fail(REMP_ERR_NOMEM, "out of host memory");
    P->shape = *shape;
    P->tables = *tables;
    std::string why;
    remp_status st = build_topo_map(*src, *shape, &P->src, &why);
    if (st == REMP_OK) st = build_topo_map(*dst, *shape, &P->dst, &why);
    if (st != REMP_OK) {
        delete P;
        return fail(st, why);
    }
    if (P->src.num_ranks() > 4096 || P->dst.num_ranks() > 4096) {
        delete P;
        return fail(REMP_ERR_INVALID_TOPOLOGY, "more than 4096 ranks");
    }
    build_items(P->src, P->dst, shape->num_layers, &P->items);

    // Both head partitions are even, so every range boundary is a multiple of g = gcd(Hl_src, Hl_dst)
    // heads: items are cut into runs of g heads (when one partition refines the other, g = min and a run is
    // a whole item), which gives every destination block the same number of equally long runs.
    P->run_heads = std::gcd(P->src.heads_per_rank, P->dst.heads_per_rank);
    P->n_sub = P->dst.heads_per_rank / P->run_heads;
    P->n_groups = (P->dst.tp / P->dst.rep) * shape->num_layers * 2;
    P->head_slice_bytes = (int64_t)shape->block_size * shape->head_dim * shape->elem_bytes;
    for (const Item& it : P->items) {
        if ((it.h_hi - it.h_lo) % P->run_heads != 0 || it.h_lo % P->run_heads != 0) {
            delete P;
            return fail(REMP_ERR_STATE, "internal: item not aligned to the run length");
        }
    }

    *out = P;
    return REMP_OK;
}

extern "C" int32_t remp_plan_num_items(const remp_plan* plan) { return plan ? (int32_t)plan->items.size() : 0; }

extern "C" remp_status remp_plan_get_items(const remp_plan* plan, int32_t* out) {
    if (!plan || !out) return fail(REMP_ERR_INVALID_ARG, "null argument");
    for (size_t i = 0; i < plan->items.size(); ++i) {
        const Item& it = plan->items[i];
        int32_t* row = out + 5 * i;
        row[0] = it.src, row[1] = it.dst, row[2] = it.layer, row[3] = it.h_lo, row[4] = it.h_hi;
    }
    return REMP_OK;
}

extern "C" remp_status remp_plan_traffic(const remp_plan* plan, int64_t total_blocks, int64_t* bytes_read,
                                         int64_t* bytes_written) {
    if (!plan || total_blocks < 0) return fail(REMP_ERR_INVALID_ARG, "null plan or negative block count");
    const remp_model_shape& m = plan->shape;
    const int64_t r = total_blocks * m.num_layers * 2 * m.num_kv_heads * plan->head_slice_bytes;
    if (bytes_read) *bytes_read = r;
    if (bytes_written) *bytes_written = r * plan->dst.rep;
    return REMP_OK;
}

extern "C" remp_status remp_plan_traffic_tokens(const remp_plan* plan, int64_t valid_tokens, int64_t* bytes_read,
                                                int64_t* bytes_written) {
    if (!plan || valid_tokens < 0) return fail(REMP_ERR_INVALID_ARG, "null plan or negative token count");
    const remp_model_shape& m = plan->shape;
    const int64_t r = valid_tokens * m.num_layers * 2 * m.num_kv_heads * (int64_t)m.head_dim * m.elem_bytes;
    if (bytes_read) *bytes_read = r;
    if (bytes_written) *bytes_written = r * plan->dst.rep;
    return REMP_OK;
}

extern "C" remp_status remp_plan_set_option(remp_plan* plan, int32_t key, int64_t value) {
    if (!plan || value < 0) return fail(REMP_ERR_INVALID_ARG, "null plan or negative option value");
    switch (key) {
        case REMP_OPT_KERNEL:
            if (value > 2) return fail(REMP_ERR_INVALID_ARG, "kernel must be 0, 1 or 2");
            plan->opt_kernel = (int)value;
            return REMP_OK;
        case REMP_OPT_CTAS_PER_SM:
            if (value > 32) return fail(REMP_ERR_INVALID_ARG, "at most 32 CTAs per SM");
            plan->opt_ctas_per_sm = (int)value;
            return REMP_OK;
        case REMP_OPT_CHUNK_BYTES:
            if (value != 0 && (value % 512 != 0 || value > 32768))
                return fail(REMP_ERR_INVALID_ARG, "chunk must be a multiple of 512 up to 32768");
            plan->opt_chunk_bytes = value;
            return REMP_OK;
        case REMP_OPT_VEC_BYTES:
            if (value != 0 && value != 16 && value != 32) return fail(REMP_ERR_INVALID_ARG, "vector width must be 16 or 32");
            plan->opt_vec_bytes = (int)value;
            return REMP_OK;
        case REMP_OPT_TILE_ITEMS:
            if (value > (1 << 30)) return fail(REMP_ERR_INVALID_ARG, "tile too large");
            plan->opt_tile_items = value;
            return REMP_OK;
        case REMP_OPT_SCHEDULE:
            if (value > 3) return fail(REMP_ERR_INVALID_ARG, "schedule must be 0..3");
            plan->opt_schedule = (int)value;
            return REMP_OK;
        case REMP_OPT_ORDER:
            if (value > 1) return fail(REMP_ERR_INVALID_ARG, "order must be 0 or 1");
            plan->opt_order = (int)value;
            return REMP_OK;
        case REMP_OPT_VALID_TOKENS_ONLY:
            plan->opt_valid_only = value ? 1 : 0;
            return REMP_OK;
        case REMP_OPT_LANES_PER_WARP:
            if (value != 0 && (value > 32 || (value & (value - 1)))) return fail(REMP_ERR_INVALID_ARG, "lanes per warp must be a power of two up to 32");
            plan->opt_lanes_per_warp = (int)value;
            return REMP_OK;
        default:
            return fail(REMP_ERR_INVALID_ARG, "unknown option");
    }
}

static remp_status status_from_word(uint32_t w) {
    if (w & kErrBadLength) return fail(REMP_ERR_BAD_LENGTH, "a sequence length is negative or wider than a table row");
    if (w & kErrOverflow) return fail(REMP_ERR_CAPACITY, "total block count does not fit 32 bits");
    if (w & kErrCapacity) return fail(REMP_ERR_CAPACITY, "live blocks do not fit the smallest destination pool");
    if (w & kErrBadBlock) return fail(REMP_ERR_BAD_BLOCK_ID, "a live block id lies outside its pool");
    if (w & kErrWaitLimit) return fail(REMP_ERR_CUDA, "an on-chip copy did not complete within the wait limit");
    return REMP_OK;
}

// ---------------------------------------------------------------------------------------------
// Device scratch of a plan: one stream-ordered allocation from a library-owned memory pool (kept warm
// between plans, so a switch costs no cudaMalloc), laid out as
//   off[num_seqs+1] | total | error word | tile counter | preempted count | pairs[pair_cap] | segs.
// Created by the first remp_alloc_dst_blocks, so planning itself needs no device.
// ---------------------------------------------------------------------------------------------

static remp_status device_pool(int device, cudaMemPool_t* out) {
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

static size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }

static void release_scratch(remp_plan* P) {
    if (!P->d_block) return;
    int cur = -1;
    cudaGetDevice(&cur);
    if (cur != P->device) cudaSetDevice(P->device);
    // Stream-ordered free: work already enqueued on last_stream may still use the block.
    if (cudaFreeAsync(P->d_block, P->last_stream) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(P->d_block);
    }
    if (cur != P->device && cur >= 0) cudaSetDevice(cur);
    P->d_block = nullptr;
    P->d_off = nullptr;
}

// A plan's scratch lives on the device that was current at its first allocation; later calls must be made
// with the same device current.
static remp_status check_device(const remp_plan* P) {
    if (P->device < 0) return REMP_OK;
    int cur = -1;
    REMP_CUDA(cudaGetDevice(&cur));
    if (cur != P->device) return fail(REMP_ERR_STATE, "the plan was used on another device; make that device current");
    return REMP_OK;
}

static remp_status ensure_scratch(remp_plan* P, int64_t need_pairs, cudaStream_t stream) {
    if (remp_status st = check_device(P)) return st;
    const int64_t n_desc = (int64_t)P->n_groups * P->n_sub;
    const int64_t n_seg = n_desc * (1 + P->dst.rep);
    if (P->d_block && need_pairs <= P->pair_cap) return REMP_OK;
    if (P->d_block) release_scratch(P);
    REMP_CUDA(cudaGetDevice(&P->device));
    REMP_CUDA(cudaDeviceGetAttribute(&P->num_sms, cudaDevAttrMultiProcessorCount, P->device));
    cudaMemPool_t pool = nullptr;
    if (remp_status st = device_pool(P->device, &pool)) return st;
    const size_t off_bytes = align16(((size_t)P->tables.num_seqs + 1 + 4) * sizeof(int32_t));
    const size_t pair_bytes = align16((size_t)need_pairs * sizeof(int4));
    const size_t seg_bytes = (size_t)n_seg * sizeof(Seg);
    REMP_CUDA(cudaMallocFromPoolAsync(&P->d_block, off_bytes + pair_bytes + seg_bytes, pool, stream));
    char* b = static_cast<char*>(P->d_block);
    P->d_off = reinterpret_cast<int32_t*>(b);
    P->d_total = P->d_off + P->tables.num_seqs + 1;
    P->d_err = reinterpret_cast<uint32_t*>(P->d_total + 1);
    P->d_counter = P->d_err + 1;
    P->d_num_preempted = P->d_counter + 1;
    P->d_pairs = reinterpret_cast<int4*>(b + off_bytes);
    P->d_segs = reinterpret_cast<Seg*>(b + off_bytes + pair_bytes);
    P->pair_cap = need_pairs;
    P->last_stream = stream;
    return REMP_OK;
}

static remp_status alloc_impl(remp_plan* plan, const int64_t* dst_capacity_blocks, int32_t base_block,
                              int32_t* dst_block_tables, int32_t* preempted, bool preempt, int64_t* total_blocks,
                              int64_t* num_preempted, cudaStream_t stream) {
    if (!plan || !dst_capacity_blocks) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (base_block < 0) return fail(REMP_ERR_INVALID_ARG, "base_block must be >= 0");
    const remp_block_tables& bt = plan->tables;
    if (!dst_block_tables && bt.num_seqs > 0 && bt.max_blocks_per_seq > 0)
        return fail(REMP_ERR_INVALID_ARG, "null dst_block_tables");
    if (preempt && !preempted && bt.num_seqs > 0) return fail(REMP_ERR_INVALID_ARG, "null preempted array");
    const int nd = plan->dst.num_ranks();
    int64_t min_cap = INT64_MAX;
    for (int r = 0; r < nd; ++r) {
        if (dst_capacity_blocks[r] < 0) return fail(REMP_ERR_INVALID_ARG, "negative destination capacity");
        min_cap = std::min(min_cap, dst_capacity_blocks[r]);
    }
    const int64_t avail = std::max<int64_t>(0, min_cap - base_block);
    // The pair list can never be longer than the table, nor than what fits the smallest pool.
    const int64_t need_pairs =
        std::max<int64_t>(1, std::min<int64_t>((int64_t)bt.num_seqs * bt.max_blocks_per_seq, avail));
    if (remp_status st = ensure_scratch(plan, need_pairs, stream)) return st;
    plan->dst_capacity.assign(dst_capacity_blocks, dst_capacity_blocks + nd);
    plan->base_block = base_block;
    plan->last_stream = stream;

    REMP_CUDA(cudaMemsetAsync(plan->d_total, 0, 4 * sizeof(int32_t), stream));  // total, error word, counters
    REMP_CUDA(launch_demand_scan(bt.seq_lens, bt.num_seqs, plan->shape.block_size, bt.max_blocks_per_seq, avail,
                                 plan->d_off, plan->d_total, plan->d_err, stream, preempt));
    REMP_CUDA(launch_remap_tables(bt.block_tables, bt.num_seqs, bt.max_blocks_per_seq, base_block, plan->d_off,
                                  dst_block_tables, plan->d_pairs, plan->d_err, stream, bt.seq_lens,
                                  plan->shape.block_size, preempt ? avail : -1, preempted, plan->d_num_preempted));
    plan->allocated = true;
    if (total_blocks || num_preempted) {
        REMP_CUDA(cudaMemcpyAsync(plan->h_result, plan->d_total, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        REMP_CUDA(cudaStreamSynchronize(stream));
        if (total_blocks) *total_blocks = plan->h_result[0];
        if (num_preempted) *num_preempted = plan->h_result[3];
        return status_from_word((uint32_t)plan->h_result[1]);
    }
    return REMP_OK;
}

extern "C" remp_status remp_alloc_dst_blocks(remp_plan* plan, const int64_t* dst_capacity_blocks, int32_t base_block,
                                             int32_t* dst_block_tables, int64_t* total_blocks, void* stream) {
    return alloc_impl(plan, dst_capacity_blocks, base_block, dst_block_tables, nullptr, false, total_blocks, nullptr,
                      static_cast<cudaStream_t>(stream));
}

extern "C" remp_status remp_alloc_dst_blocks_preempt(remp_plan* plan, const int64_t* dst_capacity_blocks,
                                                     int32_t base_block, int32_t* dst_block_tables, int32_t* preempted,
                                                     int64_t* total_blocks, int64_t* num_preempted, void* stream) {
    return alloc_impl(plan, dst_capacity_blocks, base_block, dst_block_tables, preempted, true, total_blocks,
                      num_preempted, static_cast<cudaStream_t>(stream));
}

extern "C" remp_status remp_alloc_dst_blocks_shared(remp_plan* plan, const int64_t* dst_capacity_blocks,
                                                    int32_t base_block, int64_t src_num_blocks,
                                                    int32_t* dst_block_tables, int64_t* total_blocks, void* stream_) {
    if (!plan || !dst_capacity_blocks) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (base_block < 0 || src_num_blocks < 0 || src_num_blocks > 0x7f000000LL)
        return fail(REMP_ERR_INVALID_ARG, "base_block / src_num_blocks out of range");
    const remp_block_tables& bt = plan->tables;
    if (!dst_block_tables && bt.num_seqs > 0 && bt.max_blocks_per_seq > 0)
        return fail(REMP_ERR_INVALID_ARG, "null dst_block_tables");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int nd = plan->dst.num_ranks();
    int64_t min_cap = INT64_MAX;
    for (int r = 0; r < nd; ++r) {
        if (dst_capacity_blocks[r] < 0) return fail(REMP_ERR_INVALID_ARG, "negative destination capacity");
        min_cap = std::min(min_cap, dst_capacity_blocks[r]);
    }
    const int64_t avail = std::max<int64_t>(0, min_cap - base_block);
    const int64_t entries_max = (int64_t)bt.num_seqs * bt.max_blocks_per_seq;
    if (entries_max > 0x7f000000LL) return fail(REMP_ERR_SHAPE, "block tables too large for the sharing-preserving allocator");
    const int64_t need_pairs = std::max<int64_t>(1, std::min<int64_t>(entries_max, avail));
    if (remp_status st = ensure_scratch(plan, need_pairs, stream)) return st;
    plan->dst_capacity.assign(dst_capacity_blocks, dst_capacity_blocks + nd);
    plan->base_block = base_block;
    plan->last_stream = stream;
    cudaMemPool_t pool = nullptr;
    if (remp_status st = device_pool(plan->device, &pool)) return st;
    // scratch of this call only: first[src pool] | entry_src[entries_max] | excl[entries_max]
    const size_t first_bytes = align16((size_t)std::max<int64_t>(1, src_num_blocks) * sizeof(int32_t));
    const size_t entry_bytes = align16((size_t)std::max<int64_t>(1, entries_max) * sizeof(int32_t));
    void* tmp = nullptr;
    REMP_CUDA(cudaMallocFromPoolAsync(&tmp, first_bytes + 2 * entry_bytes, pool, stream));
    int32_t* first = static_cast<int32_t*>(tmp);
    int32_t* entry_src = reinterpret_cast<int32_t*>(static_cast<char*>(tmp) + first_bytes);
    int32_t* excl = reinterpret_cast<int32_t*>(static_cast<char*>(tmp) + first_bytes + entry_bytes);

    cudaError_t e = cudaMemsetAsync(plan->d_total, 0, 4 * sizeof(int32_t), stream);
    // the demand scan gives the flat position of every entry; capacity is judged on distinct blocks later
    if (e == cudaSuccess)
        e = launch_demand_scan(bt.seq_lens, bt.num_seqs, plan->shape.block_size, bt.max_blocks_per_seq, INT64_MAX,
                               plan->d_off, plan->d_total, plan->d_err, stream, false);
    if (e == cudaSuccess)
        e = launch_dedupe(bt.block_tables, bt.num_seqs, bt.max_blocks_per_seq, base_block, plan->d_off, src_num_blocks,
                          avail, first, entry_src, excl, dst_block_tables, plan->d_pairs, plan->d_total, plan->d_err,
                          stream, plan->shape.block_size);
    cudaFreeAsync(tmp, stream);
    if (e != cudaSuccess) return cuda_fail(e, "sharing-preserving allocation");
    plan->allocated = true;
    if (total_blocks) {
        REMP_CUDA(cudaMemcpyAsync(plan->h_result, plan->d_total, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        REMP_CUDA(cudaStreamSynchronize(stream));
        *total_blocks = plan->h_result[0];
        return status_from_word((uint32_t)plan->h_result[1]);
    }
    return REMP_OK;
}

extern "C" remp_status remp_plan_status(remp_plan* plan, void* stream_) {
    if (!plan) return fail(REMP_ERR_INVALID_ARG, "null plan");
    if (!plan->d_block) return REMP_OK;  // nothing has run on the device yet
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    REMP_CUDA(cudaMemcpyAsync(plan->h_result, plan->d_total, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    REMP_CUDA(cudaStreamSynchronize(stream));
    return status_from_word((uint32_t)plan->h_result[1]);
}

namespace {

struct ShardView {  // a shard with its strides resolved
    uint64_t base;
    int64_t nb, s_layer, s_kv, s_block, s_head, s_token;
    int64_t extent;  // bytes from base to one past the last byte
};

// nl: layers of this rank that the caller's buffer holds (its whole stage, or the part inside a layer window).
remp_status resolve_shard(const remp_shard& sh, const TopoMap& T, int64_t nl, const remp_model_shape& m, ShardView* v) {
    const int64_t hs = (int64_t)m.block_size * m.head_dim * m.elem_bytes;
    const int64_t row = (int64_t)m.head_dim * m.elem_bytes;
    if (sh.num_blocks < 0) return fail(REMP_ERR_INVALID_ARG, "negative num_blocks");
    if (!sh.base && sh.num_blocks > 0) return fail(REMP_ERR_INVALID_ARG, "null shard base");
    v->base = reinterpret_cast<uint64_t>(sh.base);
    v->nb = sh.num_blocks;
    v->s_token = sh.stride_token ? sh.stride_token : row;
    v->s_head = sh.stride_head ? sh.stride_head : hs;
    // dense token rows (stride_token = head_dim*elem_bytes) fold into longer rows and need no alignment of their own
    if (v->s_token < row || v->s_head < row || (v->s_head & 15) || (v->s_token != row && ((v->s_token | row) & 15)))
        return fail(REMP_ERR_SHAPE, "stride_head and stride_token must be multiples of 16 and at least one token row");
    v->s_block = sh.stride_block ? sh.stride_block : T.heads_per_rank * hs;
    v->s_kv = sh.stride_kv ? sh.stride_kv : sh.num_blocks * v->s_block;
    v->s_layer = sh.stride_layer ? sh.stride_layer : 2 * v->s_kv;
    if (v->s_block < T.heads_per_rank * hs || v->s_kv < 0 || v->s_layer < 0)
        return fail(REMP_ERR_SHAPE, "strides must be positive and stride_block must hold all local heads");
    if ((v->base | (uint64_t)v->s_block | (uint64_t)v->s_kv | (uint64_t)v->s_layer) & 15)
        return fail(REMP_ERR_SHAPE, "shard base and strides must be multiples of 16 bytes");
    v->extent = sh.num_blocks == 0 ? 0
                                   : (nl - 1) * v->s_layer + v->s_kv + (sh.num_blocks - 1) * v->s_block +
                                         (T.heads_per_rank - 1) * v->s_head + (m.block_size - 1) * v->s_token + row;
    if (nl <= 0) v->extent = 0;
    return REMP_OK;
}

bool overlaps(const ShardView& a, const ShardView& b) {
    return a.extent && b.extent && a.base < b.base + b.extent && b.base < a.base + a.extent;
}

}  // namespace

// Build the copy descriptors of the layers [layer_lo, layer_hi), ordered (destination stage, head-owner
// group, layer, K/V, run), upload them and launch the migration kernel on `stream`.
static remp_status enqueue_migrate(remp_plan* plan, const std::vector<ShardView>& sv, const std::vector<ShardView>& dv,
                                   int layer_lo, int layer_hi, cudaStream_t stream) {
    if (remp_status st = check_device(plan)) return st;
    const remp_model_shape& m = plan->shape;
    const TopoMap &S = plan->src, &D = plan->dst;
    const int n_sub = plan->n_sub, rep = D.rep, g = plan->run_heads;
    const int64_t n_groups = (int64_t)(D.tp / rep) * (layer_hi - layer_lo) * 2;
    const int64_t n_desc = n_groups * n_sub;
    const int64_t n_seg = n_desc * (1 + rep);
    if (n_desc == 0) return REMP_OK;
    // Items arrive ordered (layer, destination TP rank, head); index their first entry per (layer, dst tp).
    if (plan->first_item.empty()) {
        plan->first_item.assign((size_t)m.num_layers * D.tp, -1);
        for (int32_t i = (int32_t)plan->items.size() - 1; i >= 0; --i)
            plan->first_item[plan->items[i].layer * D.tp + plan->items[i].dst % D.tp] = i;
    }
    const std::vector<int32_t>& first = plan->first_item;

    plan->h_segs.resize((size_t)n_seg);
    Seg* hs = plan->h_segs.data();
    Seg* hd = hs + n_desc;
    const int64_t hsb = plan->head_slice_bytes;
    // Descriptor order = order of the work along one block: with opt_order 0 a plane is (destination stage,
    // head-owner group, layer, K/V) and a block contributes the n_sub runs of that destination rank; with
    // opt_order 1 a plane is (destination stage, layer, K/V) and a block contributes the runs of ALL head-owner
    // groups, so the heads of a block are walked front to back on both sides at the same time.
    const int n_hg = D.tp / rep;
    auto fill = [&](int64_t d, int p, int hg, int l, int kv, int i) {
        const int t0 = hg * rep;  // first destination TP rank of this head-owner group
        const int h = D.head_lo[t0] + i * g;  // first head of this run
        int32_t cur = first[l * D.tp + t0];
        while (plan->items[cur].h_hi <= h) ++cur;  // the item that holds head h
        const Item& it = plan->items[cur];
        const ShardView& s = sv[it.src];
        const int lsrc = l - S.layer_start[it.src / S.tp];
        hs[d].base = s.base + lsrc * s.s_layer + kv * s.s_kv + (h - S.head_lo[it.src % S.tp]) * s.s_head;
        hs[d].bstride = s.s_block;
        hs[d].nblocks = (uint64_t)s.nb;
        hs[d].pad = 0;
        for (int r = 0; r < rep; ++r) {
            const ShardView& t = dv[D.rank(p, t0 + r)];
            Seg& o = hd[d * rep + r];
            o.base = t.base + (l - D.layer_start[p]) * t.s_layer + kv * t.s_kv + (h - D.head_lo[t0 + r]) * t.s_head;
            o.bstride = t.s_block;
            o.nblocks = (uint64_t)t.nb;
            o.pad = 0;
        }
    };
    const bool across = plan->opt_order == 1;
    int64_t d = 0;
    for (int p = 0; p < D.pp; ++p) {
        const int l_lo = std::max(layer_lo, D.layer_start[p]), l_hi = std::min(layer_hi, D.layer_start[p + 1]);
        if (across) {
            for (int l = l_lo; l < l_hi; ++l)
                for (int kv = 0; kv < 2; ++kv)
                    for (int hg = 0; hg < n_hg; ++hg)
                        for (int i = 0; i < n_sub; ++i) fill(d++, p, hg, l, kv, i);
        } else {
            for (int hg = 0; hg < n_hg; ++hg)
                for (int l = l_lo; l < l_hi; ++l)
                    for (int kv = 0; kv < 2; ++kv)
                        for (int i = 0; i < n_sub; ++i) fill(d++, p, hg, l, kv, i);
        }
    }
    // Pageable source: the runtime stages the bytes before returning, so h_segs may be reused at once.
    REMP_CUDA(cudaMemcpyAsync(plan->d_segs, hs, (size_t)n_seg * sizeof(Seg), cudaMemcpyHostToDevice, stream));

    // ---- shape of one run inside a block: g heads x block_size tokens x one token row, with the caller's
    // head/token strides. Contiguous dimensions are folded into the row; what is left is at most two strided
    // dimensions (n1 x n2 rows of row_bytes). Fully contiguous runs take the plain chunk copy.
    int64_t ssh = 0, sst = 0, dsh = 0, dst_tok = 0;
    bool have_s = false, have_d = false;
    for (const ShardView& v : sv)
        if (v.extent) {
            if (have_s && (v.s_head != ssh || v.s_token != sst))
                return fail(REMP_ERR_SHAPE, "all source shards must share stride_head and stride_token");
            ssh = v.s_head, sst = v.s_token, have_s = true;
        }
    for (const ShardView& v : dv)
        if (v.extent) {
            if (have_d && (v.s_head != dsh || v.s_token != dst_tok))
                return fail(REMP_ERR_SHAPE, "all destination shards must share stride_head and stride_token");
            dsh = v.s_head, dst_tok = v.s_token, have_d = true;
        }
    const int64_t row0 = (int64_t)m.head_dim * m.elem_bytes, bs = m.block_size;
    if (!have_s) ssh = hsb, sst = row0;
    if (!have_d) dsh = hsb, dst_tok = row0;
    int64_t row_bytes, n1, n2, s1, s2, d1, d2;
    uint32_t tok_mode = 0;  // where the token index of a row lives: 0 inside the row, 1 outer index, 2 inner index
    if (sst == row0 && dst_tok == row0) {  // token rows adjacent on both sides: a head slice is one row
        row_bytes = bs * row0, n1 = g, s1 = ssh, d1 = dsh, n2 = 1, s2 = d2 = 0;
        if (g == 1 || (ssh == row_bytes && dsh == row_bytes)) row_bytes *= g, n1 = 1;
    } else if (ssh == row0 && dsh == row0) {  // heads adjacent on both sides (token-major blocks)
        row_bytes = g * row0, n1 = bs, s1 = sst, d1 = dst_tok, n2 = 1, s2 = d2 = 0, tok_mode = 1;
        // whole token-major blocks are contiguous; in valid-tokens-only mode keep the token rows apart
        if (bs == 1 || (sst == row_bytes && dst_tok == row_bytes && !plan->opt_valid_only)) row_bytes *= bs, n1 = 1;
    } else {  // layouts differ: one (head, token) row at a time
        row_bytes = row0, n1 = g, s1 = ssh, d1 = dsh, n2 = bs, s2 = sst, d2 = dst_tok, tok_mode = 2;
    }
    const bool contiguous = n1 == 1 && n2 == 1;

    MigrateParams prm{};
    prm.src_seg = plan->d_segs;
    prm.dst_seg = plan->d_segs + n_desc;
    prm.pairs = plan->d_pairs;
    prm.total = plan->d_total;
    prm.err = plan->d_err;
    prm.tile_counter = plan->d_counter;
    prm.n_groups = (uint32_t)(across ? n_groups / n_hg : n_groups);
    prm.n_sub = (uint32_t)(across ? n_sub * n_hg : n_sub);
    prm.rep = (uint32_t)rep;
    prm.run_bytes = (uint32_t)(g * hsb);
    LaunchCfg cfg{plan->opt_kernel ? plan->opt_kernel : 1, plan->opt_ctas_per_sm, plan->num_sms,
                  plan->opt_vec_bytes ? plan->opt_vec_bytes : 16, plan->opt_lanes_per_warp ? plan->opt_lanes_per_warp : 8,
                  plan->opt_schedule == 0 ? 1 : plan->opt_schedule - 1};  // default: CTA-level dynamic tiles
    // Default chunk: 4 KiB per warp iteration (8 x 16 bytes per lane), smaller when the whole run is smaller.
    int64_t chunk = plan->opt_chunk_bytes ? plan->opt_chunk_bytes : (g * hsb <= 1024 ? 1024 : g * hsb <= 2048 ? 2048 : 4096);
    prm.chunk_bytes = (uint32_t)chunk;
    prm.nchunk = (uint32_t)((prm.run_bytes + chunk - 1) / chunk);
    prm.tile_items = (uint32_t)(plan->opt_tile_items ? plan->opt_tile_items : (cfg.dynamic == 2 ? 1 : 8));
    prm.valid_only = plan->opt_valid_only ? 1u : 0u;
    prm.block_size = (uint32_t)bs;
    prm.tok_bytes = (uint32_t)row0;
    prm.head_bytes = (uint32_t)hsb;
    if (prm.valid_only && cfg.kernel == 2) cfg.kernel = 1;  // the bulk-copy ring moves whole chunks only
    if (cfg.vec_bytes == 32) {  // 32-byte accesses need every run to start on a 32-byte boundary
        uint64_t bits = prm.run_bytes | (uint64_t)chunk;
        for (int64_t i = 0; i < n_seg; ++i) bits |= hs[i].base | (uint64_t)hs[i].bstride;
        if (bits & 31) cfg.vec_bytes = 16;
    }
    if (!contiguous) {
        // strided rows: a work item is a group of rows (rows shorter than 4 KiB) or a 4 KiB piece of one row
        cfg.kernel = 3;
        if (cfg.dynamic == 2) cfg.dynamic = 1;
        prm.chunk_bytes = 4096;
        prm.row_bytes = (uint32_t)row_bytes;
        prm.rows = (uint32_t)(n1 * n2);
        prm.n2 = (uint32_t)n2;
        prm.s1 = (uint32_t)s1, prm.s2 = (uint32_t)s2, prm.d1 = (uint32_t)d1, prm.d2 = (uint32_t)d2;
        prm.rows_per_item = (uint32_t)std::max<int64_t>(1, 4096 / row_bytes);
        prm.tok_mode = tok_mode;
        prm.nchunk = (uint32_t)((row_bytes + 4095) / 4096) * ((prm.rows + prm.rows_per_item - 1) / prm.rows_per_item);
        prm.tile_items = (uint32_t)(plan->opt_tile_items ? plan->opt_tile_items : 8);
        if (std::max({s1 * n1, s2 * n2, d1 * n1, d2 * n2}) >= ((int64_t)1 << 31))
            return fail(REMP_ERR_SHAPE, "head/token strides too large");
    }
    // The kernel indexes work items with 32 bits.
    const long double items_max = (long double)plan->pair_cap * n_desc * prm.nchunk;
    if (items_max >= 4294967295.0L) return fail(REMP_ERR_SHAPE, "more than 2^32 copy chunks; raise REMP_OPT_CHUNK_BYTES");
    plan->last_stream = stream;
    REMP_CUDA(launch_migrate(prm, cfg, stream));
    return REMP_OK;
}

extern "C" remp_status remp_migrate_kv(remp_plan* plan, const remp_shard* src, const remp_shard* dst, void* stream_) {
    if (!plan || !src || !dst) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (!plan->allocated) return fail(REMP_ERR_STATE, "remp_alloc_dst_blocks must run before remp_migrate_kv");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const remp_model_shape& m = plan->shape;
    const TopoMap &S = plan->src, &D = plan->dst;
    const int ns = S.num_ranks(), nd = D.num_ranks();

    std::vector<ShardView> sv(ns), dv(nd);
    for (int r = 0; r < ns; ++r)
        if (remp_status st = resolve_shard(src[r], S, S.stage_layers(r / S.tp), m, &sv[r])) return st;
    for (int r = 0; r < nd; ++r) {
        if (remp_status st = resolve_shard(dst[r], D, D.stage_layers(r / D.tp), m, &dv[r])) return st;
        if (dv[r].nb < plan->dst_capacity[r])
            return fail(REMP_ERR_INVALID_ARG, "a destination shard is smaller than the capacity given at allocation");
    }
    // No destination byte range may touch a source byte range (the source must stay intact).
    for (int a = 0; a < ns; ++a)
        for (int b = 0; b < nd; ++b)
            if (overlaps(sv[a], dv[b])) return fail(REMP_ERR_ALIAS, "a destination shard overlaps a source shard");
    for (int a = 0; a < nd; ++a)
        for (int b = a + 1; b < nd; ++b)
            if (overlaps(dv[a], dv[b])) return fail(REMP_ERR_ALIAS, "two destination shards overlap");

    return enqueue_migrate(plan, sv, dv, 0, m.num_layers, stream);
}

// Layer-wise streaming (section 3.4.4): the caller owns one buffer per rank that holds only the rank's layers
// inside [layer_lo, layer_hi); resolve it to a view addressed by the rank's local layer index.
extern "C" remp_status remp_migrate_kv_layers(remp_plan* plan, int32_t layer_lo, int32_t layer_hi, const remp_shard* src,
                                              const remp_shard* dst, void* stream_) {
    if (!plan || !src || !dst) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (!plan->allocated) return fail(REMP_ERR_STATE, "remp_alloc_dst_blocks must run before remp_migrate_kv_layers");
    const remp_model_shape& m = plan->shape;
    if (layer_lo < 0 || layer_hi > m.num_layers || layer_lo > layer_hi)
        return fail(REMP_ERR_INVALID_ARG, "layer window out of range");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const TopoMap &S = plan->src, &D = plan->dst;
    const int ns = S.num_ranks(), nd = D.num_ranks();
    std::vector<ShardView> sv(ns), dv(nd);
    auto window_view = [&](const remp_shard& sh, const TopoMap& T, int r, ShardView* v) -> remp_status {
        const int p = r / T.tp;
        const int lo = std::max(layer_lo, T.layer_start[p]), hi = std::min(layer_hi, T.layer_start[p + 1]);
        if (hi <= lo) {  // this rank holds no layer of the window: ignored
            *v = ShardView{};
            return REMP_OK;
        }
        if (remp_status st = resolve_shard(sh, T, hi - lo, m, v)) return st;
        v->base -= (uint64_t)((lo - T.layer_start[p]) * v->s_layer);  // index by local layer; only the window is touched
        return REMP_OK;
    };
    for (int r = 0; r < ns; ++r)
        if (remp_status st = window_view(src[r], S, r, &sv[r])) return st;
    for (int r = 0; r < nd; ++r) {
        if (remp_status st = window_view(dst[r], D, r, &dv[r])) return st;
        if (dv[r].extent && dv[r].nb < plan->dst_capacity[r])
            return fail(REMP_ERR_INVALID_ARG, "a destination shard is smaller than the capacity given at allocation");
    }
    auto span = [&](const ShardView& v, const TopoMap& T, int r) {  // the bytes of the window, for the alias check
        ShardView w = v;
        if (v.extent) w.base += (uint64_t)((std::max(layer_lo, T.layer_start[r / T.tp]) - T.layer_start[r / T.tp]) * v.s_layer);
        return w;
    };
    for (int a = 0; a < ns; ++a)
        for (int b = 0; b < nd; ++b)
            if (overlaps(span(sv[a], S, a), span(dv[b], D, b)))
                return fail(REMP_ERR_ALIAS, "a destination shard overlaps a source shard");
    for (int a = 0; a < nd; ++a)
        for (int b = a + 1; b < nd; ++b)
            if (overlaps(span(dv[a], D, a), span(dv[b], D, b))) return fail(REMP_ERR_ALIAS, "two destination shards overlap");
    return enqueue_migrate(plan, sv, dv, layer_lo, layer_hi, stream);
}

// =============================================================================================
// Host-resident caches: the same re-sharding with every buffer in host memory. Layers are streamed
// through two device staging slots in windows (host->device copy, migration kernel and device->host copy
// of consecutive windows overlap on three streams), so device memory stays at a few layers of cache no
// matter how large the cache is - the layer-wise streaming of section 3.4.4 applied to a PCIe link.
// =============================================================================================
namespace {

struct PipeGuard {  // releases everything the pipeline created, on every exit path
    cudaStream_t st[3] = {nullptr, nullptr, nullptr};
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    void* blocks[3] = {nullptr, nullptr, nullptr};
    remp_plan* plan = nullptr;
    ~PipeGuard() {
        for (cudaStream_t s : st)
            if (s) cudaStreamSynchronize(s);
        if (plan) remp_plan_destroy(plan);
        for (void* b : blocks)
            if (b) cudaFreeAsync(b, st[1]);
        for (cudaEvent_t e : ev)
            if (e) cudaEventDestroy(e);
        for (cudaStream_t s : st)
            if (s) {
                cudaStreamSynchronize(s);
                cudaStreamDestroy(s);
            }
    }
};

}  // namespace

extern "C" remp_status remp_reshard_host(const remp_topo* src, const remp_topo* dst, const remp_model_shape* shape,
                                         int32_t num_seqs, int32_t max_blocks_per_seq, const int32_t* seq_lens,
                                         const int32_t* block_tables, const remp_host_shard* src_shards,
                                         const remp_host_shard* dst_shards, int32_t base_block, int32_t window_layers,
                                         int32_t* dst_block_tables, int64_t* total_blocks, int64_t* h2d_bytes,
                                         int64_t* d2h_bytes) {
    if (!src || !dst || !shape || !src_shards || !dst_shards || !total_blocks)
        return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (num_seqs < 0 || max_blocks_per_seq < 0 || window_layers < 0)
        return fail(REMP_ERR_INVALID_ARG, "negative size");
    const size_t n_tab = (size_t)num_seqs * max_blocks_per_seq;
    if (num_seqs > 0 && (!seq_lens || (n_tab && (!block_tables || !dst_block_tables))))
        return fail(REMP_ERR_INVALID_ARG, "null table pointer");
    if (remp_status st = check_shape(*shape)) return st;

    PipeGuard G;
    int device = -1;
    REMP_CUDA(cudaGetDevice(&device));
    cudaMemPool_t pool = nullptr;
    if (remp_status st = device_pool(device, &pool)) return st;
    for (int i = 0; i < 3; ++i) REMP_CUDA(cudaStreamCreateWithFlags(&G.st[i], cudaStreamNonBlocking));
    for (int i = 0; i < 6; ++i) REMP_CUDA(cudaEventCreateWithFlags(&G.ev[i], cudaEventDisableTiming));
    cudaStream_t s_h2d = G.st[0], s_run = G.st[1], s_d2h = G.st[2];
    cudaEvent_t *ev_h2d = &G.ev[0], *ev_run = &G.ev[2], *ev_d2h = &G.ev[4];
    int64_t up = 0, down = 0;

    // ---- tables to the device, plan, destination block allocation ----
    const size_t lens_bytes = align16((size_t)num_seqs * sizeof(int32_t));
    const size_t tab_bytes = align16(n_tab * sizeof(int32_t));
    REMP_CUDA(cudaMallocFromPoolAsync(&G.blocks[0], lens_bytes + 2 * tab_bytes + 16, pool, s_run));
    char* tb = static_cast<char*>(G.blocks[0]);
    int32_t* d_lens = reinterpret_cast<int32_t*>(tb);
    int32_t* d_bt = reinterpret_cast<int32_t*>(tb + lens_bytes);
    int32_t* d_dbt = reinterpret_cast<int32_t*>(tb + lens_bytes + tab_bytes);
    if (num_seqs) REMP_CUDA(cudaMemcpyAsync(d_lens, seq_lens, (size_t)num_seqs * 4, cudaMemcpyHostToDevice, s_run));
    if (n_tab) REMP_CUDA(cudaMemcpyAsync(d_bt, block_tables, n_tab * 4, cudaMemcpyHostToDevice, s_run));
    up += (int64_t)num_seqs * 4 + (int64_t)n_tab * 4;

    remp_block_tables bt{num_seqs, max_blocks_per_seq, d_lens, d_bt};
    if (remp_status st = remp_plan_create(src, dst, shape, &bt, &G.plan)) return st;
    remp_plan* plan = G.plan;
    const TopoMap &S = plan->src, &D = plan->dst;
    const int ns = S.num_ranks(), nd = D.num_ranks();
    std::vector<int64_t> caps(nd);
    for (int r = 0; r < nd; ++r) {
        if (dst_shards[r].num_blocks < 0 || (!dst_shards[r].base && dst_shards[r].num_blocks))
            return fail(REMP_ERR_INVALID_ARG, "bad destination shard");
        caps[r] = dst_shards[r].num_blocks;
    }
    for (int r = 0; r < ns; ++r)
        if (src_shards[r].num_blocks < 0 || (!src_shards[r].base && src_shards[r].num_blocks))
            return fail(REMP_ERR_INVALID_ARG, "bad source shard");
    int64_t total = 0;
    if (remp_status st = remp_alloc_dst_blocks(plan, caps.data(), base_block, d_dbt, &total, s_run)) return st;
    *total_blocks = total;
    if (n_tab) REMP_CUDA(cudaMemcpyAsync(dst_block_tables, d_dbt, n_tab * 4, cudaMemcpyDeviceToHost, s_run));
    down += (int64_t)n_tab * 4 + 8;

    // ---- direct path: every buffer is page-locked and mapped into the device's address space, so the
    // migration kernel gathers from and scatters to host memory itself (one launch, no staging, only live
    // blocks cross the link). Taken when the caller leaves the window size to the library.
    auto mapped = [](const void* p, uint64_t* dev) {
        cudaPointerAttributes a{};
        if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        if (a.type != cudaMemoryTypeHost || !a.devicePointer) return false;
        *dev = reinterpret_cast<uint64_t>(a.devicePointer);
        return true;
    };
    if (window_layers == 0 && total > 0) {
        std::vector<ShardView> sv(ns), dv(nd);
        bool direct = true;
        const int64_t row = (int64_t)shape->head_dim * shape->elem_bytes, hs = plan->head_slice_bytes;
        auto view = [&](const remp_host_shard& sh, const TopoMap& T, int r, ShardView* v) {
            *v = ShardView{};
            if (sh.num_blocks == 0) return true;
            if (!mapped(sh.base, &v->base)) return false;
            v->nb = sh.num_blocks;
            v->s_token = row, v->s_head = hs;
            v->s_block = T.heads_per_rank * hs;
            v->s_kv = v->nb * v->s_block;
            v->s_layer = 2 * v->s_kv;
            v->extent = T.stage_layers(r / T.tp) * v->s_layer;
            return (v->base & 15) == 0;
        };
        for (int r = 0; r < ns && direct; ++r)
            if ((r % S.tp) % S.rep == 0) direct = view(src_shards[r], S, r, &sv[r]);  // replicas are never read
        for (int r = 0; r < nd && direct; ++r) direct = view(dst_shards[r], D, r, &dv[r]);
        if (direct) {
            if (remp_status st = enqueue_migrate(plan, sv, dv, 0, shape->num_layers, s_run)) return st;
            int64_t moved_r = 0, moved_w = 0;
            remp_plan_traffic(plan, total, &moved_r, &moved_w);
            for (int i = 0; i < 3; ++i) REMP_CUDA(cudaStreamSynchronize(G.st[i]));
            if (h2d_bytes) *h2d_bytes = up + moved_r;
            if (d2h_bytes) *d2h_bytes = down + moved_w;
            return remp_plan_status(plan, s_run);
        }
    }

    // ---- windows: sub-ranges of the common refinement of both stage partitions ----
    const int L = shape->num_layers;
    const int64_t hsb = plan->head_slice_bytes;
    auto layer_bytes = [&](const TopoMap& T, const remp_host_shard* sh, int rank) {
        return 2 * sh[rank].num_blocks * T.heads_per_rank * hsb;
    };
    int64_t src_row = 0, dst_row = 0;  // largest per-layer footprint of one stage row of ranks
    for (int p = 0; p < S.pp; ++p) {
        int64_t b = 0;
        for (int t = 0; t < S.tp; ++t) b += layer_bytes(S, src_shards, S.rank(p, t));
        src_row = std::max(src_row, b);
    }
    for (int p = 0; p < D.pp; ++p) {
        int64_t b = 0;
        for (int t = 0; t < D.tp; ++t) b += layer_bytes(D, dst_shards, D.rank(p, t));
        dst_row = std::max(dst_row, b);
    }
    int W = window_layers;
    if (W == 0) W = (int)std::max<int64_t>(1, std::min<int64_t>(L, ((int64_t)1 << 30) / std::max<int64_t>(1, src_row)));
    std::vector<std::pair<int, int>> windows;
    for (int l = 0; l < L;) {
        const int stop = std::min(S.layer_start[S.stage_of_layer[l] + 1], D.layer_start[D.stage_of_layer[l] + 1]);
        const int hi = std::min(l + W, stop);
        windows.emplace_back(l, hi);
        l = hi;
    }
    if (total > 0 && src_row > 0 && dst_row > 0) {
        const size_t s_slot = align16((size_t)src_row * W), d_slot = align16((size_t)dst_row * W);
        REMP_CUDA(cudaMallocFromPoolAsync(&G.blocks[1], 2 * s_slot, pool, s_run));
        REMP_CUDA(cudaMallocFromPoolAsync(&G.blocks[2], 2 * d_slot, pool, s_run));
        REMP_CUDA(cudaEventRecord(ev_run[0], s_run));  // staging exists from here on
        REMP_CUDA(cudaStreamWaitEvent(s_h2d, ev_run[0], 0));
        std::vector<ShardView> sv(ns), dv(nd);
        for (size_t w = 0; w < windows.size(); ++w) {
            const int l0 = windows[w].first, l1 = windows[w].second, nl = l1 - l0, slot = (int)(w & 1);
            const int ps = S.stage_of_layer[l0], pd = D.stage_of_layer[l0];
            char* s_base = static_cast<char*>(G.blocks[1]) + slot * s_slot;
            char* d_base = static_cast<char*>(G.blocks[2]) + slot * d_slot;
            std::fill(sv.begin(), sv.end(), ShardView{});
            std::fill(dv.begin(), dv.end(), ShardView{});
            // host -> device: the window's layers of every source rank of stage ps
            if (w >= 2) REMP_CUDA(cudaStreamWaitEvent(s_h2d, ev_run[slot], 0));  // slot read by window w-2
            int64_t o = 0;
            for (int t = 0; t < S.tp; ++t) {
                const int r = S.rank(ps, t);
                const int64_t lb = layer_bytes(S, src_shards, r);
                const int64_t first = l0 - S.layer_start[ps];
                if (t % S.rep != 0) continue;  // only the lowest-numbered replica of a head is ever read
                if (lb) {
                    REMP_CUDA(cudaMemcpyAsync(s_base + o, static_cast<const char*>(src_shards[r].base) + first * lb,
                                              (size_t)(nl * lb), cudaMemcpyHostToDevice, s_h2d));
                    up += nl * lb;
                }
                ShardView& v = sv[r];
                v.nb = src_shards[r].num_blocks;
                v.s_token = (int64_t)shape->head_dim * shape->elem_bytes;
                v.s_head = hsb;
                v.s_block = S.heads_per_rank * hsb;
                v.s_kv = v.nb * v.s_block;
                v.s_layer = lb;
                v.extent = nl * lb;
                v.base = reinterpret_cast<uint64_t>(s_base + o) - (uint64_t)(first * lb);
                o += nl * lb;
            }
            REMP_CUDA(cudaEventRecord(ev_h2d[slot], s_h2d));
            // migrate the window
            o = 0;
            std::vector<int64_t> d_off(D.tp);
            for (int t = 0; t < D.tp; ++t) {
                const int r = D.rank(pd, t);
                const int64_t lb = layer_bytes(D, dst_shards, r);
                const int64_t first = l0 - D.layer_start[pd];
                ShardView& v = dv[r];
                v.nb = dst_shards[r].num_blocks;
                v.s_token = (int64_t)shape->head_dim * shape->elem_bytes;
                v.s_head = hsb;
                v.s_block = D.heads_per_rank * hsb;
                v.s_kv = v.nb * v.s_block;
                v.s_layer = lb;
                v.extent = nl * lb;
                v.base = reinterpret_cast<uint64_t>(d_base + o) - (uint64_t)(first * lb);
                d_off[t] = o;
                o += nl * lb;
            }
            REMP_CUDA(cudaStreamWaitEvent(s_run, ev_h2d[slot], 0));
            if (w >= 2) REMP_CUDA(cudaStreamWaitEvent(s_run, ev_d2h[slot], 0));  // slot drained by window w-2
            if (remp_status st = enqueue_migrate(plan, sv, dv, l0, l1, s_run)) return st;
            REMP_CUDA(cudaEventRecord(ev_run[slot], s_run));
            // device -> host: only the allocated block range of every (layer, K/V) plane
            REMP_CUDA(cudaStreamWaitEvent(s_d2h, ev_run[slot], 0));
            for (int t = 0; t < D.tp; ++t) {
                const int r = D.rank(pd, t);
                const int64_t blk = D.heads_per_rank * hsb, plane = dst_shards[r].num_blocks * blk;
                const int64_t first = l0 - D.layer_start[pd];
                for (int64_t pl = 0; pl < 2 * (int64_t)nl; ++pl) {
                    const int64_t in_plane = base_block * blk;
                    REMP_CUDA(cudaMemcpyAsync(
                        static_cast<char*>(dst_shards[r].base) + (2 * first + pl) * plane + in_plane,
                        d_base + d_off[t] + pl * plane + in_plane, (size_t)(total * blk), cudaMemcpyDeviceToHost, s_d2h));
                    down += total * blk;
                }
            }
            REMP_CUDA(cudaEventRecord(ev_d2h[slot], s_d2h));
        }
    }
    for (int i = 0; i < 3; ++i) REMP_CUDA(cudaStreamSynchronize(G.st[i]));
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return remp_plan_status(plan, s_run);
}
