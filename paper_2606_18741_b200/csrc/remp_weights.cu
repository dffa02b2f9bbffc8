// Model weights from a host store (section 3.3 of the paper, "Shared Model Weight Store"): the full model state
// sits once in host memory, and the GPU shard of every target rank is rebuilt from it - PP picks the layers of
// the rank's stage, TP slices the partitioned tensors, replicated tensors are taken whole.
// Host part: the packed shard layout and the slice list. Device part: one gather kernel that reads the slices
// straight out of page-locked host memory over the host link (16-byte loads, 4 KiB per warp iteration, tiles
// drawn from a device counter) and writes the shards; pageable stores go through the copy engine instead.

#include <algorithm>

#include "remp_internal.h"

namespace remp {
namespace {

constexpr int64_t kSliceAlign = 256;

struct Slice {  // one tensor slice of one rank: rows x row_bytes out of a [rows_full][pitch] host array
    int32_t rank, param, layer;  // layer = -1 for first/last-stage parameters
    int64_t src_off;             // bytes from the parameter's host_base
    int64_t pitch;               // bytes between consecutive source rows
    int64_t dst_off;             // bytes from the rank's shard base
    int64_t rows, row_bytes;     // local extent
};

remp_status check_param(const remp_weight_param& w, int i) {
    auto bad = [&](const char* what) { return fail(REMP_ERR_SHAPE, "weight parameter " + std::to_string(i) + ": " + what); };
    if (!w.host_base) return fail(REMP_ERR_INVALID_ARG, "weight parameter " + std::to_string(i) + ": null host_base");
    if (w.rows < 1 || w.cols < 1) return bad("rows and cols must be positive");
    if (w.elem_bytes != 1 && w.elem_bytes != 2 && w.elem_bytes != 4) return bad("elem_bytes must be 1, 2 or 4");
    if (w.partition < REMP_W_REPLICATED || w.partition > REMP_W_SPLIT_ROW_GROUPS) return bad("unknown partition");
    if (w.scope < REMP_W_EVERY_LAYER || w.scope > REMP_W_LAST_STAGE) return bad("unknown scope");
    if (w.partition == REMP_W_SPLIT_ROW_GROUPS && (w.groups < 1 || w.rows % w.groups != 0))
        return bad("groups must divide rows");
    if ((reinterpret_cast<uint64_t>(w.host_base) & 15) || (w.scope == REMP_W_EVERY_LAYER && (w.layer_stride & 15)))
        return bad("host_base and layer_stride must be multiples of 16 bytes");
    if (w.scope == REMP_W_EVERY_LAYER && w.layer_stride < w.rows * w.cols * w.elem_bytes)
        return bad("layer_stride is smaller than one instance");
    return REMP_OK;
}

// Local extent of parameter w on TP rank t of tp ranks: rows [r0, r0 + nr), columns [c0, c0 + nc).
remp_status local_extent(const remp_weight_param& w, int tp, int t, int i, int64_t* r0, int64_t* nr, int64_t* c0, int64_t* nc) {
    *r0 = 0, *nr = w.rows, *c0 = 0, *nc = w.cols;
    auto bad = [&](const char* what) {
        return fail(REMP_ERR_INVALID_TOPOLOGY, "weight parameter " + std::to_string(i) + ": " + what);
    };
    switch (w.partition) {
        case REMP_W_REPLICATED: break;
        case REMP_W_SPLIT_ROWS:
            if (w.rows % tp) return bad("TP must divide the rows of a row-split parameter");
            *nr = w.rows / tp, *r0 = t * *nr;
            break;
        case REMP_W_SPLIT_COLS:
            if (w.cols % tp) return bad("TP must divide the columns of a column-split parameter");
            *nc = w.cols / tp, *c0 = t * *nc;
            break;
        case REMP_W_SPLIT_ROW_GROUPS: {  // groups dealt like KV heads: even split, or one group shared by TP/groups ranks
            const int64_t gsz = w.rows / w.groups;
            if (tp <= w.groups) {
                if (w.groups % tp) return bad("TP must divide the number of row groups, or be a multiple of it");
                *nr = (w.groups / tp) * gsz, *r0 = t * *nr;
            } else {
                if (tp % w.groups) return bad("TP must divide the number of row groups, or be a multiple of it");
                *nr = gsz, *r0 = (t / (tp / w.groups)) * gsz;
            }
            break;
        }
    }
    if (((*nc * w.elem_bytes) & 15) || ((*c0 * w.elem_bytes) & 15) || ((w.cols * w.elem_bytes) & 15))
        return fail(REMP_ERR_SHAPE, "weight parameter " + std::to_string(i) +
                                        ": rows of a slice must start and end on 16-byte boundaries");
    return REMP_OK;
}

// The packed layout of every rank in [rank_lo, rank_hi): its slices in shard order and the shard size.
remp_status build_slices(const remp_topo& topo, int L, const remp_weight_param* params, int n_params, int rank_lo,
                         int rank_hi, std::vector<Slice>* out, std::vector<int64_t>* shard_bytes) {
    if (!params || n_params < 0 || L < 1) return fail(REMP_ERR_INVALID_ARG, "null parameter list or no layers");
    if (topo.tp < 1) return fail(REMP_ERR_INVALID_TOPOLOGY, "TP and PP must be >= 1");
    std::vector<int> layer_start;
    std::string why;
    if (remp_status st = build_layer_start(topo, L, &layer_start, &why)) return fail(st, why);
    for (int i = 0; i < n_params; ++i)
        if (remp_status st = check_param(params[i], i)) return st;
    if (rank_lo < 0 || rank_hi > topo.tp * topo.pp || rank_lo > rank_hi) return fail(REMP_ERR_INVALID_ARG, "rank out of range");
    out->clear();
    shard_bytes->assign((size_t)(rank_hi - rank_lo), 0);
    for (int rank = rank_lo; rank < rank_hi; ++rank) {
        const int p = rank / topo.tp, t = rank % topo.tp;
        int64_t off = 0;
        auto add = [&](int i, int layer) -> remp_status {
            const remp_weight_param& w = params[i];
            int64_t r0, nr, c0, nc;
            if (remp_status st = local_extent(w, topo.tp, t, i, &r0, &nr, &c0, &nc)) return st;
            Slice s;
            s.rank = rank, s.param = i, s.layer = layer;
            s.pitch = w.cols * w.elem_bytes;
            s.src_off = (layer > 0 ? layer * w.layer_stride : 0) + r0 * s.pitch + c0 * w.elem_bytes;
            s.dst_off = off;
            s.rows = nr, s.row_bytes = nc * w.elem_bytes;
            out->push_back(s);
            off += (nr * s.row_bytes + kSliceAlign - 1) / kSliceAlign * kSliceAlign;
            return REMP_OK;
        };
        if (p == 0)
            for (int i = 0; i < n_params; ++i)
                if (params[i].scope == REMP_W_FIRST_STAGE)
                    if (remp_status st = add(i, -1)) return st;
        for (int l = layer_start[p]; l < layer_start[p + 1]; ++l)
            for (int i = 0; i < n_params; ++i)
                if (params[i].scope == REMP_W_EVERY_LAYER)
                    if (remp_status st = add(i, l)) return st;
        if (p == topo.pp - 1)
            for (int i = 0; i < n_params; ++i)
                if (params[i].scope == REMP_W_LAST_STAGE)
                    if (remp_status st = add(i, -1)) return st;
        (*shard_bytes)[(size_t)(rank - rank_lo)] = off;
    }
    return REMP_OK;
}

// ---- device side ----
struct alignas(16) GatherSlice {
    uint64_t src, dst;       // first byte of the slice on either side (src: host memory as the device sees it)
    uint64_t pitch;          // bytes between source rows
    uint32_t row_bytes;      // bytes of a local row (a multiple of 16)
    uint32_t rows;
    uint32_t pieces_per_row;  // 4 KiB pieces a long row is cut into (rows_per_item == 1), else 1
    uint32_t rows_per_item;   // whole rows one item takes when a row is shorter than 4 KiB
    uint64_t first_item;      // index of the slice's first work item
};

constexpr int kGatherThreads = 256;

// Work item = up to 4 KiB of one slice: a piece of a long row, or several whole short rows. A warp gathers
// the item with 16-byte loads from host memory (all in flight before the first store) and writes it densely.
__global__ void __launch_bounds__(kGatherThreads) weight_gather_kernel(const GatherSlice* __restrict__ slices,
                                                                      uint32_t n_slices, uint64_t n_items,
                                                                      unsigned long long* __restrict__ counter,
                                                                      uint32_t tile_items) {
    __shared__ unsigned long long next_tile[2];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) next_tile[0] = blockIdx.x;
    __syncthreads();
    for (uint32_t buf = 0;; buf ^= 1) {
        const uint64_t t0 = next_tile[buf] * tile_items;
        if (t0 >= n_items) break;
        if (threadIdx.x == 0) next_tile[buf ^ 1] = gridDim.x + atomicAdd(counter, 1ull);
        const uint64_t t1 = min(n_items, t0 + tile_items);
        for (uint64_t w = t0 + warp; w < t1; w += kGatherThreads / 32) {
            uint32_t lo = 0, hi = n_slices;  // the last slice whose first item is at or before w
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (__ldg(&slices[mid].first_item) <= w) lo = mid; else hi = mid;
            }
            const GatherSlice s = slices[lo];
            const uint32_t q = (uint32_t)(w - s.first_item);
            const uint32_t vpr = s.row_bytes >> 4;  // vectors per local row
            uint4 v[8];
            uint32_t doff[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t x = u * 32 + lane;  // vector of the item
                uint32_t row, col;
                bool ok;
                if (s.rows_per_item > 1) {
                    const uint32_t ri = x / vpr;
                    row = q * s.rows_per_item + ri, col = x - ri * vpr;
                    ok = ri < s.rows_per_item && row < s.rows;
                } else {
                    row = q / s.pieces_per_row;
                    col = (q - row * s.pieces_per_row) * 256 + x;
                    ok = col < vpr;
                }
                doff[u] = ok ? row * s.row_bytes + col * 16 : 0xffffffffu;  // a slice is below 4 GiB (checked on the host)
                if (ok) {
                    const char* sp = reinterpret_cast<const char*>(s.src + (uint64_t)row * s.pitch + col * 16);
                    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                                 : "l"(sp));
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (doff[u] != 0xffffffffu)
                    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(s.dst + doff[u]), "r"(v[u].x),
                                 "r"(v[u].y), "r"(v[u].z), "r"(v[u].w)
                                 : "memory");
        }
        __syncthreads();
    }
    // the last CTA to finish puts the scheduler word back to zero (tiles drawn in the low half, CTAs done in the high)
    if (threadIdx.x == 0) {
        const unsigned long long old = atomicAdd(counter, 1ull << 32);
        if ((uint32_t)(old >> 32) == gridDim.x - 1) atomicExch(counter, 0ull);
    }
}

bool device_view(const void* host, uint64_t* dev) {
    cudaPointerAttributes a{};
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return false;
    *dev = reinterpret_cast<uint64_t>(a.devicePointer);
    return true;
}

}  // namespace
}  // namespace remp

using namespace remp;

extern "C" int64_t remp_weight_shard_bytes(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                                           int32_t num_params, int32_t rank) {
    if (!topo) return fail(REMP_ERR_INVALID_ARG, "null topology");
    std::vector<Slice> slices;
    std::vector<int64_t> bytes;
    if (remp_status st = build_slices(*topo, num_layers, params, num_params, rank, rank + 1, &slices, &bytes)) return st;
    return bytes[0];
}

extern "C" remp_status remp_weight_slice(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                                         int32_t num_params, int32_t rank, int32_t param, int32_t layer, int64_t* offset,
                                         int64_t* rows, int64_t* cols) {
    if (!topo || !offset || !rows || !cols) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (param < 0 || param >= num_params) return fail(REMP_ERR_INVALID_ARG, "parameter index out of range");
    std::vector<Slice> slices;
    std::vector<int64_t> bytes;
    if (remp_status st = build_slices(*topo, num_layers, params, num_params, rank, rank + 1, &slices, &bytes)) return st;
    const int want_layer = params[param].scope == REMP_W_EVERY_LAYER ? layer : -1;
    for (const Slice& s : slices)
        if (s.param == param && s.layer == want_layer) {
            *offset = s.dst_off, *rows = s.rows, *cols = s.row_bytes / params[param].elem_bytes;
            return REMP_OK;
        }
    return fail(REMP_ERR_INVALID_ARG, "the rank does not hold this parameter (other stage or layer)");
}

extern "C" remp_status remp_weights_reshard(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                                            int32_t num_params, void* const* dst_shards, int64_t* h2d_bytes,
                                            int32_t max_ctas, void* stream_) {
    if (!topo || !dst_shards) return fail(REMP_ERR_INVALID_ARG, "null argument");
    if (max_ctas < 0) return fail(REMP_ERR_INVALID_ARG, "negative max_ctas");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<Slice> slices;
    std::vector<int64_t> bytes;
    const int nr = topo->tp * topo->pp;
    if (remp_status st = build_slices(*topo, num_layers, params, num_params, 0, nr, &slices, &bytes)) return st;
    for (int r = 0; r < nr; ++r) {
        if (bytes[(size_t)r] > 0 && !dst_shards[r]) return fail(REMP_ERR_INVALID_ARG, "null destination shard");
        if (reinterpret_cast<uint64_t>(dst_shards[r]) & (kSliceAlign - 1))
            return fail(REMP_ERR_SHAPE, "destination shards must be 256-byte aligned");
    }
    int64_t moved = 0;
    for (const Slice& s : slices) {
        moved += s.rows * s.row_bytes;
        if (s.rows * s.row_bytes >= ((int64_t)1 << 32)) return fail(REMP_ERR_SHAPE, "a weight slice of 4 GiB or more");
    }
    if (h2d_bytes) *h2d_bytes = moved;
    if (slices.empty()) return REMP_OK;

    // Is the whole store visible to the device (page-locked, mapped)? Then one kernel gathers everything.
    std::vector<uint64_t> dev_base((size_t)num_params, 0);
    bool mapped = true;
    for (int i = 0; i < num_params && mapped; ++i) mapped = device_view(params[i].host_base, &dev_base[(size_t)i]);
    if (!mapped) {
        // copy engine: one strided copy per slice (pageable memory is staged by the runtime, synchronously)
        for (const Slice& s : slices)
            REMP_CUDA(cudaMemcpy2DAsync(static_cast<char*>(dst_shards[s.rank]) + s.dst_off, (size_t)s.row_bytes,
                                        static_cast<const char*>(params[s.param].host_base) + s.src_off, (size_t)s.pitch,
                                        (size_t)s.row_bytes, (size_t)s.rows, cudaMemcpyHostToDevice, stream));
        return REMP_OK;
    }

    std::vector<GatherSlice> gs(slices.size());
    uint64_t items = 0;
    for (size_t k = 0; k < slices.size(); ++k) {
        const Slice& s = slices[k];
        GatherSlice& g = gs[k];
        g.src = dev_base[(size_t)s.param] + (uint64_t)s.src_off;
        g.dst = reinterpret_cast<uint64_t>(dst_shards[s.rank]) + (uint64_t)s.dst_off;
        g.pitch = (uint64_t)s.pitch;
        g.row_bytes = (uint32_t)s.row_bytes;
        g.rows = (uint32_t)s.rows;
        g.rows_per_item = (uint32_t)std::max<int64_t>(1, 4096 / s.row_bytes);
        g.pieces_per_row = g.rows_per_item > 1 ? 1u : (uint32_t)((s.row_bytes + 4095) / 4096);
        g.first_item = items;
        items += g.rows_per_item > 1 ? (uint64_t)((s.rows + g.rows_per_item - 1) / g.rows_per_item)
                                     : (uint64_t)s.rows * g.pieces_per_row;
    }
    int device = -1, sms = 0;
    REMP_CUDA(cudaGetDevice(&device));
    REMP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    cudaMemPool_t pool = nullptr;
    if (remp_status st = device_pool(device, &pool)) return st;
    void* scratch = nullptr;  // scheduler word | slice records, returned to the pool in stream order
    const size_t rec_bytes = gs.size() * sizeof(GatherSlice);
    REMP_CUDA(cudaMallocFromPoolAsync(&scratch, 16 + rec_bytes, pool, stream));
    cudaError_t e = cudaMemsetAsync(scratch, 0, 16, stream);
    // the runtime stages a pageable source before it returns, so `gs` may go out of scope
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(static_cast<char*>(scratch) + 16, gs.data(), rec_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) {
        const uint32_t tile = 8;
        const uint64_t tiles = (items + tile - 1) / tile;
        const uint64_t fill = max_ctas > 0 ? (uint64_t)max_ctas : (uint64_t)sms * 4;
        const int grid = (int)std::max<uint64_t>(1, std::min<uint64_t>(fill, tiles));
        weight_gather_kernel<<<grid, kGatherThreads, 0, stream>>>(
            reinterpret_cast<const GatherSlice*>(static_cast<char*>(scratch) + 16), (uint32_t)gs.size(), items,
            static_cast<unsigned long long*>(scratch), tile);
        count_launch();
        e = cudaGetLastError();
    }
    cudaFreeAsync(scratch, stream);
    if (e != cudaSuccess) return cuda_fail(e, "weight gather");
    return REMP_OK;
}
