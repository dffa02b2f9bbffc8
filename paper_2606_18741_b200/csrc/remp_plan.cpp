// Host planner of libremp: topology maps (section 3.4.1), the Algorithm-1 item list, plan objects and their
// introspection. Nothing here touches the device.

#include <algorithm>
#include <new>
#include <numeric>

#include "remp_internal.h"

namespace remp {

// ---------------------------------------------------------------------------------------------
// Topology maps (section 3.4.1). Layers: contiguous ascending stages. Heads: even contiguous split,
// or one head per rank with rep consecutive ranks per head when TP exceeds the head count.
// ---------------------------------------------------------------------------------------------
// pp_owner: PP contiguous ascending layer ranges; even split with the first (L mod PP) stages one layer longer, or
// the caller's explicit boundaries.
remp_status build_layer_start(const remp_topo& t, int L, std::vector<int>* layer_start, std::string* why) {
    if (t.pp < 1 || t.pp > L) {
        *why = t.pp < 1 ? "TP and PP must be >= 1" : "PP exceeds the number of layers";
        return REMP_ERR_INVALID_TOPOLOGY;
    }
    layer_start->assign(t.pp + 1, 0);
    if (t.pp_layer_start) {
        for (int p = 0; p <= t.pp; ++p) (*layer_start)[p] = t.pp_layer_start[p];
        bool ok = (*layer_start)[0] == 0 && (*layer_start)[t.pp] == L;
        for (int p = 0; p < t.pp && ok; ++p) ok = (*layer_start)[p + 1] > (*layer_start)[p];
        if (!ok) {
            *why = "pp_layer_start must rise strictly from 0 to num_layers";
            return REMP_ERR_INVALID_TOPOLOGY;
        }
    } else {
        const int q = L / t.pp, r = L % t.pp;
        for (int p = 0; p < t.pp; ++p) (*layer_start)[p + 1] = (*layer_start)[p] + q + (p < r ? 1 : 0);
    }
    return REMP_OK;
}

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
    if (remp_status st = build_layer_start(t, L, &T.layer_start, why)) return st;
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

remp_status check_shape(const remp_model_shape& m) {
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

extern "C" remp_status remp_rank_ownership(const remp_topo* topo, const remp_model_shape* shape, int32_t rank,
                                           int32_t* out) {
    if (!topo || !shape || !out) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (remp_status st = check_shape(*shape)) return st;
    TopoMap T;
    std::string why;
    if (remp_status st = build_topo_map(*topo, *shape, &T, &why)) return fail(st, why);
    if (rank < 0 || rank >= T.num_ranks()) return fail(REMP_ERR_INVALID_ARG, "rank out of range");
    const int p = rank / T.tp, t = rank % T.tp;
    out[0] = T.layer_start[p], out[1] = T.layer_start[p + 1];
    out[2] = T.head_lo[t], out[3] = T.head_lo[t] + T.heads_per_rank;
    return REMP_OK;
}

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

extern "C" remp_status remp_plan_partition(const remp_plan* plan, const int32_t* src_rank_device,
                                           const int32_t* dst_rank_device, int32_t device, int32_t* recv_items,
                                           int32_t* num_recv, int32_t* send_items, int32_t* num_send) {
    if (!plan || !src_rank_device || !dst_rank_device || !num_recv || !num_send || device < 0)
        return fail(REMP_ERR_INVALID_ARG, "null argument or negative device");
    for (int r = 0; r < plan->src.num_ranks(); ++r)
        if (src_rank_device[r] < 0) return fail(REMP_ERR_INVALID_ARG, "negative device index");
    for (int r = 0; r < plan->dst.num_ranks(); ++r)
        if (dst_rank_device[r] < 0) return fail(REMP_ERR_INVALID_ARG, "negative device index");
    int32_t nr = 0, nsend = 0;
    auto put = [](int32_t* rows, int32_t n, const Item& it, int32_t other) {
        if (!rows) return;
        int32_t* row = rows + 6 * (int64_t)n;
        row[0] = it.src, row[1] = it.dst, row[2] = it.layer, row[3] = it.h_lo, row[4] = it.h_hi, row[5] = other;
    };
    for (const Item& it : plan->items) {
        const int32_t sd = src_rank_device[it.src], dd = dst_rank_device[it.dst];
        if (dd == device) put(recv_items, nr++, it, sd);
        if (sd == device && dd != device) put(send_items, nsend++, it, dd);
    }
    *num_recv = nr;
    *num_send = nsend;
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
            if (value > 2) return fail(REMP_ERR_INVALID_ARG, "order must be 0, 1 or 2");
            plan->opt_order = (int)value;
            return REMP_OK;
        case REMP_OPT_VALID_TOKENS_ONLY:
            plan->opt_valid_only = value ? 1 : 0;
            return REMP_OK;
        case REMP_OPT_LANES_PER_WARP:
            if (value != 0 && (value > 32 || (value & (value - 1)))) return fail(REMP_ERR_INVALID_ARG, "lanes per warp must be a power of two up to 32");
            plan->opt_lanes_per_warp = (int)value;
            return REMP_OK;
        case REMP_OPT_ALLOC_PATH:
            if (value > 2) return fail(REMP_ERR_INVALID_ARG, "allocation path must be 0, 1 or 2");
            plan->opt_alloc_path = (int)value;
            return REMP_OK;
        case REMP_OPT_WAIT_SPINS:
            if (value > (1 << 20) + 1) return fail(REMP_ERR_INVALID_ARG, "wait limit too large");
            plan->opt_wait_spins = value;
            return REMP_OK;
        default:
            return fail(REMP_ERR_INVALID_ARG, "unknown option");
    }
}

