// remp_reshard_host: the re-sharding for caches that live in host memory.

#include <algorithm>

#include "remp_internal.h"

using namespace remp;

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
    // The same rule as remp_migrate_kv, on the host buffers: no destination shard may touch a source shard or
    // another destination shard (the source must stay intact, and every destination byte has one writer).
    {
        const int64_t blk = plan->head_slice_bytes;
        auto span = [&](const remp_host_shard& sh, const TopoMap& T, int r, uint64_t* lo, uint64_t* hi) {
            *lo = reinterpret_cast<uint64_t>(sh.base);
            *hi = *lo + (uint64_t)(T.stage_layers(r / T.tp) * 2 * sh.num_blocks * T.heads_per_rank * blk);
        };
        auto meet = [](uint64_t a0, uint64_t a1, uint64_t b0, uint64_t b1) { return a0 < a1 && b0 < b1 && a0 < b1 && b0 < a1; };
        for (int b = 0; b < nd; ++b) {
            uint64_t d0, d1, o0, o1;
            span(dst_shards[b], D, b, &d0, &d1);
            for (int a = 0; a < ns; ++a) {
                span(src_shards[a], S, a, &o0, &o1);
                if (meet(d0, d1, o0, o1)) return fail(REMP_ERR_ALIAS, "a destination shard overlaps a source shard");
            }
            for (int a = b + 1; a < nd; ++a) {
                span(dst_shards[a], D, a, &o0, &o1);
                if (meet(d0, d1, o0, o1)) return fail(REMP_ERR_ALIAS, "two destination shards overlap");
            }
        }
    }
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
    // Measured on a PCIe 5 link: the kernel reading and writing host memory moves about 40 GB/s each way at once,
    // two copy engines about 46 GB/s each - but a contiguous copy carries the unused blocks of the source pools
    // along. So the staged path only wins when the pools are almost full.
    int64_t max_src_blocks = 0;
    for (int r = 0; r < ns; ++r) max_src_blocks = std::max(max_src_blocks, src_shards[r].num_blocks);
    const bool pools_nearly_full = total > 0 && (double)max_src_blocks <= 1.06 * (double)total;
    if (window_layers == 0 && total > 0 && !pools_nearly_full) {
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
