// Device-facing host code of libremp: plan scratch, destination block allocation (plain, capacity-constrained,
// sharing-preserving), shard resolution, the addressing tables of a launch and the migration launches (whole cache,
// layer windows, destination ranks spread over several GPUs).

#include <algorithm>
#include <cstring>

#include "remp_internal.h"

namespace remp {

remp_status status_from_word(uint32_t w) {
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
//   status words (total, error word, preempted count, 64-bit tile-scheduler word) | off[num_seqs+1] | scan tile
//   sums | pairs | addressing tables (only when they are too large for the kernel parameters).
// Created by the first remp_alloc_dst_blocks, so planning itself needs no device.
// ---------------------------------------------------------------------------------------------

void release_scratch(remp_plan_s* P) {
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

// Largest size the addressing tables of this plan can take: a view per rank, a record per layer, a plane
// group per (destination stage, head-owner group) and the sentinel.
static size_t table_bytes_max(const remp_plan_s* P) {
    const size_t views = (size_t)(P->src.num_ranks() + P->dst.num_ranks()) * sizeof(RankView);
    const size_t layers = align16((size_t)P->shape.num_layers * sizeof(LayerSrc));
    const size_t groups = ((size_t)P->dst.pp * (P->dst.tp / P->dst.rep) + 1) * sizeof(PlaneGroup);
    return views + layers + groups;
}

remp_status ensure_scratch(remp_plan_s* P, int64_t need_pairs, cudaStream_t stream) {
    if (remp_status st = check_device(P)) return st;
    if (P->d_block && need_pairs <= P->pair_cap) return REMP_OK;
    if (P->d_block) release_scratch(P);
    REMP_CUDA(cudaGetDevice(&P->device));
    REMP_CUDA(cudaDeviceGetAttribute(&P->num_sms, cudaDevAttrMultiProcessorCount, P->device));
    cudaMemPool_t pool = nullptr;
    if (remp_status st = device_pool(P->device, &pool)) return st;
    const size_t word_bytes = align16(kNumWords * sizeof(int32_t));
    const size_t off_bytes = word_bytes + align16(((size_t)P->tables.num_seqs + 1) * sizeof(int32_t));
    const size_t tile_bytes = align16(((size_t)P->tables.num_seqs / 1024 + 1) * sizeof(long long));
    const size_t pair_bytes = align16((size_t)need_pairs * sizeof(int4));
    const size_t tab_max = table_bytes_max(P);
    const size_t tab_bytes = tab_max > kTabBytes ? align16(tab_max) : 0;
    REMP_CUDA(cudaMallocFromPoolAsync(&P->d_block, off_bytes + tile_bytes + pair_bytes + tab_bytes, pool, stream));
    char* b = static_cast<char*>(P->d_block);
    P->d_total = reinterpret_cast<int32_t*>(b) + kWordTotal;
    P->d_err = reinterpret_cast<uint32_t*>(b) + kWordErr;
    P->d_num_preempted = reinterpret_cast<uint32_t*>(b) + kWordPreempted;
    P->d_sched = reinterpret_cast<unsigned long long*>(reinterpret_cast<int32_t*>(b) + kWordSched);
    P->d_off = reinterpret_cast<int32_t*>(b + word_bytes);
    P->d_tile_sums = reinterpret_cast<long long*>(b + off_bytes);
    P->d_pairs = reinterpret_cast<int4*>(b + off_bytes + tile_bytes);
    P->d_tab = tab_bytes ? reinterpret_cast<uint8_t*>(b + off_bytes + tile_bytes + pair_bytes) : nullptr;
    P->tab_cap = (int64_t)tab_bytes;
    P->pair_cap = need_pairs;
    P->last_stream = stream;
    return REMP_OK;
}

}  // namespace remp

using namespace remp;

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
    // ids are 32-bit: blocks at or beyond 2^31 - base_block cannot be named, so they do not count as capacity
    const int64_t avail = std::min<int64_t>(std::max<int64_t>(0, min_cap - base_block), 0x7fffffffLL - base_block);
    // The pair list can never be longer than the table, nor than what fits the smallest pool.
    const int64_t need_pairs =
        std::max<int64_t>(1, std::min<int64_t>((int64_t)bt.num_seqs * bt.max_blocks_per_seq, avail));
    const bool fused_ok =
        bt.num_seqs <= kFusedMaxSeqs && (int64_t)bt.num_seqs * bt.max_blocks_per_seq <= kFusedMaxEntries;
    if (plan->opt_alloc_path == 1 && !fused_ok)
        return fail(REMP_ERR_INVALID_ARG, "the single-launch allocation takes at most 1024 sequences and 2^18 table entries");
    if (remp_status st = ensure_scratch(plan, need_pairs, stream)) return st;
    plan->dst_capacity.assign(dst_capacity_blocks, dst_capacity_blocks + nd);
    plan->base_block = base_block;
    plan->last_stream = stream;

    if (fused_ok && plan->opt_alloc_path != 2) {
        // small inputs: scan, table rewrite and the reset of every status word in one cluster launch
        REMP_CUDA(launch_alloc_fused(bt.seq_lens, bt.block_tables, bt.num_seqs, bt.max_blocks_per_seq,
                                     plan->shape.block_size, base_block, avail, preempt, plan->d_off, plan->d_total,
                                     dst_block_tables, plan->d_pairs, preempted, stream));
    } else {
        REMP_CUDA(cudaMemsetAsync(plan->d_total, 0, kNumWords * sizeof(int32_t), stream));  // all status words
        REMP_CUDA(launch_demand_scan(bt.seq_lens, bt.num_seqs, plan->shape.block_size, bt.max_blocks_per_seq, avail,
                                     plan->d_off, plan->d_total, plan->d_err, stream, preempt, plan->d_tile_sums));
        REMP_CUDA(launch_remap_tables(bt.block_tables, bt.num_seqs, bt.max_blocks_per_seq, base_block, plan->d_off,
                                      dst_block_tables, plan->d_pairs, plan->d_err, stream, bt.seq_lens,
                                      plan->shape.block_size, preempt ? avail : -1, preempted, plan->d_num_preempted));
    }
    plan->allocated = true;
    if (total_blocks || num_preempted) {
        REMP_CUDA(cudaMemcpyAsync(plan->h_result, plan->d_total, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        REMP_CUDA(cudaStreamSynchronize(stream));
        if (total_blocks) *total_blocks = plan->h_result[0];
        if (num_preempted) *num_preempted = plan->h_result[kWordPreempted];
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
    const int64_t avail = std::min<int64_t>(std::max<int64_t>(0, min_cap - base_block), 0x7fffffffLL - base_block);
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

    cudaError_t e = cudaMemsetAsync(plan->d_total, 0, kNumWords * sizeof(int32_t), stream);
    // the demand scan gives the flat position of every entry; capacity is judged on distinct blocks later
    if (e == cudaSuccess)
        e = launch_demand_scan(bt.seq_lens, bt.num_seqs, plan->shape.block_size, bt.max_blocks_per_seq, INT64_MAX,
                               plan->d_off, plan->d_total, plan->d_err, stream, false, plan->d_tile_sums);
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

namespace remp {

// Build the addressing tables of the layers [layer_lo, layer_hi) - planes ordered (destination stage, head-owner
// group, layer, K/V), or (destination stage, layer, K/V) with all head-owner groups of a block together - and
// launch the migration kernel on `stream`. The tables ride in the kernel parameters; nothing is uploaded unless
// there are so many ranks that they do not fit.
remp_status enqueue_migrate(remp_plan_s* plan, const std::vector<ShardView>& sv, const std::vector<ShardView>& dv,
                            int layer_lo, int layer_hi, cudaStream_t stream, const std::vector<uint8_t>* dst_here) {
    if (remp_status st = check_device(plan)) return st;
    const remp_model_shape& m = plan->shape;
    const TopoMap &S = plan->src, &D = plan->dst;
    const int n_sub = plan->n_sub, rep = D.rep, g = plan->run_heads;
    const int64_t n_groups = (int64_t)(D.tp / rep) * (layer_hi - layer_lo) * 2;
    const int64_t n_desc = n_groups * n_sub;
    if (n_desc == 0) return REMP_OK;
    if (m.num_layers > 65535) return fail(REMP_ERR_SHAPE, "more than 65535 layers");
    const int64_t hsb = plan->head_slice_bytes;
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
    // Short contiguous runs (a power of two up to 2 KiB, whole blocks, default kernel): the contiguous kernel takes
    // the run of several consecutive blocks as one item of up to 4 KiB. Other contiguous runs of at most 1 KiB (a third
    // of 4 KiB when not a power of two; or partial blocks) go through the row kernel, which packs several blocks into an item
    // as well (768-byte runs: 0.84 of the copy rate one block per item).
    const bool one_piece = n1 == 1 && n2 == 1;
    const bool pow2_run = (row_bytes & (row_bytes - 1)) == 0;
    const bool block_groups = one_piece && pow2_run && row_bytes <= 2048 && !plan->opt_valid_only &&
                              plan->opt_kernel != 2 && plan->opt_vec_bytes != 32 && !plan->opt_chunk_bytes;
    const bool contiguous = one_piece && (row_bytes > (pow2_run ? 1024 : 4096 / 3) || block_groups);

    // Order of the work along one block: rank by rank, a plane is (destination stage, head-owner group, layer,
    // K/V) and a block contributes the n_sub runs of that destination rank; across ranks, a plane is (destination
    // stage, layer, K/V) and a block contributes the runs of ALL head-owner groups, so the heads of a block are
    // walked front to back on both sides at the same time.
    const int n_hg = D.tp / rep;
    // Rows shorter than a 128-byte line that are pieces of wider source rows (token-major blocks split between
    // ranks): walking all destination ranks of a block together lets the pieces of a line be read while it is
    // still in L2 (64-byte rows: 4.6 -> 6.0 TB/s); otherwise one rank after the other is as fast or faster.
    // (the same for contiguous head slices below 128 bytes when a source block holds more heads than one run: 64-byte
    // slices 0.66 -> 0.88 of the copy rate)
    // (and for strided rows below 1 KiB that are not a power of two - 192-byte rows of head_dim 96: 0.80 -> 1.00,
    // 640-byte rows 0.93 -> 0.97; rows of 128, 256 or 512 bytes lose 1 % that way and stay rank by rank)
    const bool split_lines = contiguous ? row_bytes < 128 && (int64_t)S.heads_per_rank * hsb > row_bytes
                                        : sst > row_bytes && (row_bytes < 128 || (!pow2_run && row_bytes < 1024));
    // (with destination ranks on other GPUs the work goes rank by rank, so that whole planes can be left out)
    const bool across = !dst_here && (plan->opt_order == 1 || (plan->opt_order == 0 && split_lines && n_hg > 1));

    // ---- addressing tables: source views | destination views | LayerSrc per layer | plane groups + sentinel ----
    const int ns = S.num_ranks(), nd = D.num_ranks();
    const size_t off_dst = (size_t)ns * sizeof(RankView);
    const size_t off_layer = off_dst + (size_t)nd * sizeof(RankView);
    const size_t off_group = off_layer + align16((size_t)m.num_layers * sizeof(LayerSrc));
    std::vector<PlaneGroup> groups;
    uint32_t planes = 0;
    for (int p = 0; p < D.pp; ++p) {
        const int l_lo = std::max(layer_lo, D.layer_start[p]), l_hi = std::min(layer_hi, D.layer_start[p + 1]);
        if (l_hi <= l_lo) continue;
        for (int hg = 0; hg < (across ? 1 : n_hg); ++hg) {
            if (dst_here) {  // a head-owner group none of whose replicas lives here is another GPU's work
                bool any = false;
                for (int r = 0; r < rep; ++r) any = any || (*dst_here)[(size_t)D.rank(p, hg * rep + r)];
                if (!any) continue;
            }
            groups.push_back(PlaneGroup{planes, (uint16_t)l_lo, (uint16_t)(l_lo - D.layer_start[p]),
                                        (uint16_t)D.rank(p, 0), (uint16_t)(hg * D.heads_per_rank)});
            planes += (uint32_t)(l_hi - l_lo) * 2;
        }
    }
    const uint32_t n_pg = (uint32_t)groups.size();
    groups.push_back(PlaneGroup{planes, 0, 0, 0, 0});
    const size_t tab_bytes = off_group + groups.size() * sizeof(PlaneGroup);
    plan->h_tab.assign(align16(tab_bytes), 0);
    uint8_t* tb = plan->h_tab.data();
    auto put_view = [](uint8_t* at, const ShardView& v) {
        const RankView r{v.extent ? v.base : 0, v.s_layer, v.s_kv, v.s_block, v.extent ? (uint64_t)v.nb : 0};
        memcpy(at, &r, sizeof r);
    };
    for (int r = 0; r < ns; ++r) put_view(tb + (size_t)r * sizeof(RankView), sv[r]);
    for (int r = 0; r < nd; ++r) {
        put_view(tb + off_dst + (size_t)r * sizeof(RankView), dv[r]);
        if (dst_here && !(*dst_here)[(size_t)r]) {
            const RankView elsewhere{kViewElsewhere, 0, 0, 0, 0};
            memcpy(tb + off_dst + (size_t)r * sizeof(RankView), &elsewhere, sizeof elsewhere);
        }
    }
    if (planes == 0) return REMP_OK;  // nothing of this window lands on this GPU
    for (int l = 0; l < m.num_layers; ++l) {
        const int ps = S.stage_of_layer[l];
        const LayerSrc ls{(uint16_t)S.rank(ps, 0), (uint16_t)(l - S.layer_start[ps])};
        memcpy(tb + off_layer + (size_t)l * sizeof(LayerSrc), &ls, sizeof ls);
    }
    memcpy(tb + off_group, groups.data(), groups.size() * sizeof(PlaneGroup));

    MigrateParams prm{};
    prm.pairs = plan->d_pairs;
    prm.total = plan->d_total;
    prm.err = plan->d_err;
    prm.sched = plan->d_sched;
    prm.tab_bytes = (uint32_t)tab_bytes;
    prm.off_dst = (uint32_t)off_dst, prm.off_layer = (uint32_t)off_layer, prm.off_group = (uint32_t)off_group;
    prm.n_pg = n_pg;
    prm.run_heads = (uint32_t)g;
    prm.hl_src = (uint32_t)S.heads_per_rank, prm.hl_dst = (uint32_t)D.heads_per_rank;
    prm.rep_src = (uint32_t)S.rep;
    auto log2_or_32 = [](uint32_t x) {
        uint32_t sh = 0;
        while ((1u << sh) < x) ++sh;
        return (1u << sh) == x ? sh : 32u;
    };
    prm.hl_src_shift = log2_or_32(prm.hl_src), prm.hl_dst_shift = log2_or_32(prm.hl_dst);
    prm.sh_src = ssh, prm.sh_dst = dsh;
    prm.wait_spins = plan->opt_wait_spins ? (uint32_t)(plan->opt_wait_spins - 1) : (1u << 20);
    prm.n_groups = planes;
    prm.n_sub = (uint32_t)(across ? n_sub * n_hg : n_sub);
    prm.rep = (uint32_t)rep;
    prm.run_bytes = (uint32_t)(g * hsb);
    LaunchCfg cfg{plan->opt_kernel ? plan->opt_kernel : 1, plan->opt_ctas_per_sm, plan->num_sms,
                  plan->opt_vec_bytes ? plan->opt_vec_bytes : 16, plan->opt_lanes_per_warp ? plan->opt_lanes_per_warp : 8,
                  plan->opt_schedule == 0 ? 1 : plan->opt_schedule - 1, 0};  // default: CTA-level dynamic tiles
    // Default chunk: 4 KiB per warp iteration (8 x 16 bytes per lane), smaller when the whole run is smaller
    // (32-byte vectors start at 1 KiB chunks).
    int64_t chunk = plan->opt_chunk_bytes ? plan->opt_chunk_bytes : (g * hsb <= 512 ? 512 : g * hsb <= 1024 ? 1024 : g * hsb <= 2048 ? 2048 : 4096);
    prm.chunk_bytes = (uint32_t)chunk;
    prm.nchunk = (uint32_t)((prm.run_bytes + chunk - 1) / chunk);
    // A tile is at least 16 KiB of work (8 chunks of 4 KiB for the usual runs): small runs take more chunks per
    // tile so that the tile counter is not hit more than once per 16 KiB moved.
    const int64_t item_bytes = std::min<int64_t>(chunk, g * hsb);
    const int64_t tile_bytes = item_bytes <= 512 ? 65536 : 16384;  // tiny items: amortise the hand-over further
    const int64_t auto_tile = std::max<int64_t>(8, ((tile_bytes + item_bytes - 1) / item_bytes + 7) / 8 * 8);
    prm.tile_items = (uint32_t)(plan->opt_tile_items ? plan->opt_tile_items : (cfg.dynamic == 2 ? 1 : auto_tile));
    prm.valid_only = plan->opt_valid_only ? 1u : 0u;
    // partial blocks move fewer bytes per item: larger tiles keep the per-tile work (position decode, hand-over) small
    if (prm.valid_only && !plan->opt_tile_items && cfg.dynamic != 2) prm.tile_items *= 2;
    prm.block_size = (uint32_t)bs;
    prm.tok_bytes = (uint32_t)row0;
    prm.head_bytes = (uint32_t)hsb;
    if (prm.valid_only && cfg.kernel == 2) cfg.kernel = 1;  // the bulk-copy ring moves whole chunks only
    if (cfg.vec_bytes == 32 && chunk < 1024) cfg.vec_bytes = 16;
    if (prm.valid_only) cfg.vec_bytes = 16;  // token rows are only known to be multiples of 16 bytes
    if (cfg.vec_bytes == 32) {  // 32-byte accesses need every run to start on a 32-byte boundary
        uint64_t bits = prm.run_bytes | (uint64_t)chunk | (uint64_t)ssh | (uint64_t)dsh;
        for (const std::vector<ShardView>* side : {&sv, &dv})
            for (const ShardView& v : *side)
                if (v.extent) bits |= v.base | (uint64_t)v.s_layer | (uint64_t)v.s_kv | (uint64_t)v.s_block;
        if (bits & 31) cfg.vec_bytes = 16;
    }
    if (cfg.kernel == 1 && contiguous && !regcopy_chunk_supported(chunk, cfg.vec_bytes))
        return fail(REMP_ERR_INVALID_ARG, "the register-copy kernel takes chunks of 512, 1024, 2048, 4096 or 8192 bytes "
                                          "(at least 1024 with 32-byte vectors)");
    if (block_groups) {
        // an item = the run of B consecutive live blocks, B * run_bytes <= 4 KiB, B <= 32 (one pair record per lane)
        cfg.kernel = 4;
        const uint32_t B = (uint32_t)std::min<int64_t>(32, 4096 / row_bytes);
        prm.blocks_per_item = B;
        prm.bpi_shift = log2_or_32(B);
        prm.run_shift = log2_or_32((uint32_t)(row_bytes >> 4));
        prm.nchunk = 1;
        prm.chunk_bytes = (uint32_t)std::max<int64_t>(512, B * row_bytes);  // bytes of one item: 512 .. 4096
        const int64_t tile = std::max<int64_t>(8, (16384 / prm.chunk_bytes + 7) / 8 * 8);
        prm.tile_items = (uint32_t)(plan->opt_tile_items ? plan->opt_tile_items : (cfg.dynamic == 2 ? 1 : tile));
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
        prm.tok_mode = tok_mode;
        prm.vpr_shift = log2_or_32(prm.row_bytes >> 4);
        prm.n2_shift = log2_or_32(prm.n2);
        auto magic = [](uint32_t d) { return d > 1 ? (uint32_t)((1ull << 32) / d + 1) : 0u; };  // divisions by shift or multiply
        prm.vpr_magic = magic(prm.row_bytes >> 4), prm.n2_magic = magic(prm.n2);
        // a whole run of at most 1 KiB (a third of 4 KiB when not a power of two: 1280-byte runs 0.82 -> 0.98 of the
        // copy rate in groups of three, while groups of two measured slower than single blocks): one
        // item takes the run of several consecutive live blocks (up to 4 KiB, at
        // most 32 blocks) - one block per item leaves a warp with too few bytes in flight (512-byte runs of 64-byte
        // rows: 0.83 of the copy rate one by one, 1.03 in groups of eight)
        const int64_t run_total = (int64_t)prm.rows * row_bytes;
        const bool group_blocks = run_total <= 1024 || (run_total * 3 <= 4096 && (run_total & (run_total - 1)) != 0);
        prm.blocks_per_item = group_blocks ? (uint32_t)std::min<int64_t>(32, 4096 / run_total) : 1;
        prm.run_shift = log2_or_32((uint32_t)(run_total >> 4));
        prm.run_magic = magic((uint32_t)(run_total >> 4));
        // an item is 4 KiB (256 vectors) of the run's rows taken back to back
        const int64_t run_vecs = (int64_t)prm.rows * (row_bytes >> 4);
        prm.nchunk = (uint32_t)((run_vecs + 255) / 256);
        if (run_vecs * (row_bytes >> 4) >= ((int64_t)1 << 32))  // keeps the kernel's divisions by multiplication exact
            return fail(REMP_ERR_SHAPE, "a run of more than 2^32 / (row_bytes / 16) vectors");
        const int64_t row_item_bytes = std::min<int64_t>(4096, (int64_t)prm.rows * row_bytes * prm.blocks_per_item);
        // one-block items below 4 KiB (2 KiB runs): the per-tile work (hand-over, barrier, position decode) weighs
        // more, so a tile holds 32 KiB
        const int64_t row_tile_bytes = prm.blocks_per_item == 1 && row_item_bytes < 4096 ? 32768 : 16384;
        prm.tile_items = (uint32_t)(plan->opt_tile_items
                                        ? plan->opt_tile_items
                                        : std::max<int64_t>(8, ((row_tile_bytes + row_item_bytes - 1) / row_item_bytes + 7) / 8 * 8) *
                                              (prm.valid_only ? 2 : 1));  // partial blocks move fewer bytes per item
        if (std::max({s1 * n1, s2 * n2, d1 * n1, d2 * n2}) >= ((int64_t)1 << 31))
            return fail(REMP_ERR_SHAPE, "head/token strides too large");
    }
    // The kernel indexes work items with 32 bits.
    const long double items_max = (long double)plan->pair_cap * n_desc * prm.nchunk;
    if (items_max >= 4290000000.0L) return fail(REMP_ERR_SHAPE, "more than 2^32 copy chunks; raise REMP_OPT_CHUNK_BYTES");
    // no launch needs more CTAs than it can have tiles (the pair list's capacity bounds the live blocks)
    const long double per_item_blocks = cfg.kernel >= 3 && prm.blocks_per_item > 1 ? prm.blocks_per_item : 1;
    cfg.max_tiles = (int64_t)(items_max / per_item_blocks / std::max<uint32_t>(1, prm.tile_items)) + 1;
    {  // the digits of the two strides a warp may step by, for the run structure of this launch
        const bool multi = cfg.kernel >= 3 && prm.blocks_per_item > 1;
        const uint32_t pieces = multi ? 1u : prm.nchunk, per_block = prm.n_sub * pieces;
        auto digits = [&](uint32_t stride) {
            StepDigits d;
            d.dk = stride / per_block;
            const uint32_t dr = stride - d.dk * per_block;
            d.di = dr / pieces;
            d.dch = dr - d.di * pieces;
            return d;
        };
        prm.warps_per_cta = 8;
        prm.step1 = digits(1), prm.step_warps = digits(prm.warps_per_cta);
    }
    plan->last_stream = stream;
    // Tables that fit ride in the kernel parameters; larger ones (hundreds of ranks) are uploaded. The runtime
    // stages a pageable source before it returns, so h_tab may be reused at once.
    TabPool pool;
    if (tab_bytes <= kTabBytes) {
        memcpy(&pool, tb, align16(tab_bytes));
        prm.gtab = nullptr;
    } else {
        if (!plan->d_tab || (int64_t)tab_bytes > plan->tab_cap) return fail(REMP_ERR_STATE, "internal: table scratch too small");
        REMP_CUDA(cudaMemcpyAsync(plan->d_tab, tb, tab_bytes, cudaMemcpyHostToDevice, stream));
        prm.gtab = plan->d_tab;
    }
    REMP_CUDA(launch_migrate(prm, pool, cfg, stream));
    return REMP_OK;
}

}  // namespace remp

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


// Destination ranks spread over several GPUs (sections 3.4.2 and 3.4.3): this GPU executes the items whose
// destination rank is mapped to it, reading remote sources in place.
extern "C" remp_status remp_migrate_kv_exchange(remp_plan* plan, const int32_t* src_rank_device,
                                                const int32_t* dst_rank_device, int32_t device, const remp_shard* src,
                                                const remp_shard* dst, void* stream_) {
    if (!plan || !src_rank_device || !dst_rank_device || !src || !dst || device < 0)
        return fail(REMP_ERR_INVALID_ARG, "null argument or negative device");
    if (!plan->allocated) return fail(REMP_ERR_STATE, "remp_alloc_dst_blocks must run before remp_migrate_kv_exchange");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const remp_model_shape& m = plan->shape;
    const TopoMap &S = plan->src, &D = plan->dst;
    const int ns = S.num_ranks(), nd = D.num_ranks();
    std::vector<uint8_t> here((size_t)nd, 0), needed((size_t)ns, 0);
    bool remote_source = false;
    for (const Item& it : plan->items) {
        if (dst_rank_device[it.dst] != device) continue;
        here[(size_t)it.dst] = 1;
        needed[(size_t)it.src] = 1;
        if (src_rank_device[it.src] < 0) return fail(REMP_ERR_INVALID_ARG, "negative device index");
        remote_source = remote_source || src_rank_device[it.src] != device;
    }
    if (remote_source && plan->opt_kernel == 2)
        return fail(REMP_ERR_INVALID_ARG, "the bulk-copy kernel is not used with sources on another GPU");
    std::vector<ShardView> sv((size_t)ns), dv((size_t)nd);
    for (int r = 0; r < ns; ++r)
        if (needed[(size_t)r])
            if (remp_status st = resolve_shard(src[r], S, S.stage_layers(r / S.tp), m, &sv[(size_t)r])) return st;
    for (int r = 0; r < nd; ++r) {
        if (!here[(size_t)r]) continue;
        if (remp_status st = resolve_shard(dst[r], D, D.stage_layers(r / D.tp), m, &dv[(size_t)r])) return st;
        if (dv[(size_t)r].nb < plan->dst_capacity[(size_t)r])
            return fail(REMP_ERR_INVALID_ARG, "a destination shard is smaller than the capacity given at allocation");
    }
    for (int a = 0; a < ns; ++a)
        for (int b = 0; b < nd; ++b)
            if (overlaps(sv[(size_t)a], dv[(size_t)b])) return fail(REMP_ERR_ALIAS, "a destination shard overlaps a source shard");
    for (int a = 0; a < nd; ++a)
        for (int b = a + 1; b < nd; ++b)
            if (overlaps(dv[(size_t)a], dv[(size_t)b])) return fail(REMP_ERR_ALIAS, "two destination shards overlap");
    return enqueue_migrate(plan, sv, dv, 0, m.num_layers, stream, &here);
}
