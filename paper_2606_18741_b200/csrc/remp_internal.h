// Internal declarations shared by the host planner and the CUDA kernels of libremp.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "remp.h"

struct remp_plan_s;

namespace remp {

// ---- device error word (bit set) -------------------------------------------------------------
enum : uint32_t {
    kErrCapacity = 1u << 0,   // base + total > smallest destination pool
    kErrBadLength = 1u << 1,  // negative length or demand wider than a table row
    kErrOverflow = 1u << 2,   // total block count does not fit int32
    kErrBadBlock = 1u << 3,   // a live table entry outside the source (or destination) pool
    kErrWaitLimit = 1u << 4,  // a bounded wait on an on-chip copy barrier ran out
    kErrFatalMask = kErrCapacity | kErrBadLength | kErrOverflow  // nothing may be copied
};

// ---- topology maps (section 3.4.1: pp_owner, tp_owner, rank) ----------------------------------
struct TopoMap {
    int tp = 0, pp = 0;
    int heads_per_rank = 0;  // Hl
    int rep = 1;             // ranks sharing one head (TP > H)
    std::vector<int> layer_start;     // [pp+1]
    std::vector<int> stage_of_layer;  // [L]
    std::vector<int> head_lo;         // [tp]
    std::vector<int> first_owner;     // [H] lowest TP rank holding head h

    int num_ranks() const { return tp * pp; }
    int rank(int p, int t) const { return p * tp + t; }
    int stage_layers(int p) const { return layer_start[p + 1] - layer_start[p]; }
};

remp_status build_layer_start(const remp_topo& t, int L, std::vector<int>* layer_start, std::string* why);
remp_status build_topo_map(const remp_topo& t, const remp_model_shape& m, TopoMap* out, std::string* why);

// Status words of a plan, in this order at the start of its scratch (the scheduler word is 8-byte aligned).
enum { kWordTotal = 0, kWordErr = 1, kWordPreempted = 2, kWordSched = 4, kNumWords = 6 };

struct Item {  // one RecvItem of Algorithm 1 (the block set B is the plan-wide live set)
    int32_t src, dst, layer, h_lo, h_hi;
};

// ---- device-side addressing tables ------------------------------------------------------------
// The migration kernel turns (destination plane, run) into a source and a destination address with a few small
// tables instead of one record per run: their size depends on the number of ranks and layers only (about
// 1 KiB for the 70B shape), so they travel inside the kernel's parameters and a switch uploads nothing.
struct RankView {      // one rank's pool as the kernel sees it (strides in bytes)
    uint64_t base;     // address of (local layer 0, K, block 0, local head 0)
    int64_t s_layer, s_kv, s_block;
    uint64_t nb;       // pool size in blocks, for the bounds check
};
constexpr uint64_t kViewElsewhere = ~0ull;  // RankView.base of a destination rank that lives on another GPU: skipped
struct LayerSrc {      // per layer: where the source side keeps it
    uint16_t rank0;    // first rank of the source stage that owns the layer (stage * TP_src)
    uint16_t lloc;     // index of the layer inside that stage
};
struct PlaneGroup {    // a run of consecutive destination planes (layer, K/V) that share everything else
    uint32_t first_plane;  // planes [first_plane, next group's first_plane), two per layer (K then V)
    uint16_t layer0;       // global index of the group's first layer
    uint16_t lloc0;        // index of that layer inside the destination stage
    uint16_t rank0;        // first rank of the destination stage (stage * TP_dst)
    uint16_t head0;        // first head of run 0 of the group's planes
};
constexpr uint32_t kTabBytes = 4096;  // tables up to this size ride in the kernel parameters
struct TabPool {
    uint4 q[kTabBytes / 16];
};

// How far one step of `stride` work items moves the position (block, run, piece of the run) of a work item:
// stride = dk * (runs * pieces) + di * pieces + dch.
struct StepDigits {
    uint32_t dk, di, dch;
};

struct MigrateParams {
    const int4* pairs;     // [NB_live] (source block, destination block, valid tokens, unused)
    const int32_t* total;  // NB_live, written by the allocation kernels
    uint32_t* err;
    // dynamic tile scheduler, one 64-bit word: low half = tiles drawn so far, high half = CTAs that have finished.
    // The last CTA to finish puts the word back to zero, so it is zero between launches.
    unsigned long long* sched;
    // addressing tables: source views | destination views | LayerSrc per layer | PlaneGroups + one sentinel.
    // gtab = NULL: the tables are the TabPool parameter; else a device copy (more ranks than the pool holds)
    const uint8_t* gtab;
    uint32_t tab_bytes, off_dst, off_layer, off_group, n_pg;
    uint32_t run_heads;        // heads per run
    uint32_t hl_src, hl_dst;   // heads per rank on either side
    uint32_t hl_src_shift, hl_dst_shift;  // their log2 when powers of two, else 32
    uint32_t rep_src;          // source ranks that share a head (the lowest one is read)
    int64_t sh_src, sh_dst;    // head strides inside a block
    uint32_t n_groups;     // destination planes
    uint32_t n_sub;        // runs per destination block within a plane
    uint32_t rep;          // destination replicas per run
    uint32_t run_bytes;    // contiguous bytes per (run, block)
    uint32_t chunk_bytes;  // bytes moved per warp iteration / ring stage
    uint32_t nchunk;       // ceil(run_bytes / chunk_bytes)
    uint32_t tile_items;   // consecutive work items a CTA takes at a time (register-copy kernel)
    // strided-row kernel only: a run is `rows` rows of row_bytes, row r at (r / n2) * s1 + (r % n2) * s2 in the
    // source and (r / n2) * d1 + (r % n2) * d2 in the destination; nchunk counts the items of one run
    uint32_t row_bytes, rows, n2, s1, s2, d1, d2;
    uint32_t vpr_shift, n2_shift;  // log2 of (row_bytes / 16) and of n2 when they are powers of two, else 32
    uint32_t vpr_magic, n2_magic, run_magic;  // else floor(2^32 / d) + 1: x / d == __umulhi(x, magic) while x * d < 2^32
    uint32_t blocks_per_item;      // > 1 when a whole run is shorter than 4 KiB: consecutive blocks share an item
    uint32_t bpi_shift;            // log2(blocks_per_item) in the multi-block mode of the contiguous kernel
    uint32_t run_shift;            // log2 of the 16-byte vectors of one run when a power of two, else 32
    // valid-tokens-only mode: of a block whose pair says valid < block_size only the first `valid` tokens move
    uint32_t valid_only, block_size, tok_bytes, head_bytes;
    uint32_t tok_mode;  // strided rows: 0 tokens lie inside a row, 1 the token is the outer row index, 2 the inner
    uint32_t wait_spins;  // bulk-copy kernel: try_wait calls before a copy barrier is given up
    StepDigits step1, step_warps;  // a step of 1 item and of one item per warp of the CTA (see Stepper)
    uint32_t warps_per_cta;
};

struct LaunchCfg {
    int kernel;       // 1 register copy, 2 bulk ring, 3 strided rows, 4 register copy with multi-block items (3 and 4
                      // are chosen by the library)
    int ctas_per_sm;  // 0 = default
    int num_sms;
    int vec_bytes;       // register copy: 16 or 32
    int lanes_per_warp;  // bulk ring: stage-owning lanes per warp
    int dynamic;         // register copy: 1 = tiles drawn from a global counter
    int64_t max_tiles;   // upper bound of the tiles of this launch (from the pair-list capacity): caps the grid
};

// Kernel launchers (remp_kernels.cu). All only enqueue on `stream`.
cudaError_t launch_demand_scan(const int32_t* seq_lens, int32_t num_seqs, int32_t block_size, int32_t max_blocks,
                               int64_t avail_blocks, int32_t* off, int32_t* total, uint32_t* err, cudaStream_t stream,
                               bool preempt = false, long long* tile_scratch = nullptr);
cudaError_t launch_remap_tables(const int32_t* block_tables, int32_t num_seqs, int32_t max_blocks, int32_t base_block,
                                const int32_t* off, int32_t* dst_block_tables, int4* pairs, uint32_t* err,
                                cudaStream_t stream, const int32_t* seq_lens, int32_t block_size,
                                int64_t keep_below = -1, int32_t* preempted = nullptr,
                                uint32_t* num_preempted = nullptr);
// Fused allocation for at most kFusedMaxSeqs sequences (one launch, no memset): demand, prefix sum, capacity check,
// table rewrite, pair list; also leaves total, error word, preempted count and both tile-scheduler counters
// in their start state. Returns cudaErrorNotSupported when the input is outside its range (use the calls above).
constexpr int32_t kFusedMaxSeqs = 1024;
constexpr int64_t kFusedMaxEntries = 1 << 18;
cudaError_t launch_alloc_fused(const int32_t* seq_lens, const int32_t* block_tables, int32_t num_seqs,
                               int32_t max_blocks, int32_t block_size, int32_t base_block, int64_t avail_blocks,
                               bool preempt, int32_t* off, int32_t* words, int32_t* dst_block_tables, int4* pairs,
                               int32_t* preempted, cudaStream_t stream);
// tab: the addressing tables when p.gtab is NULL (p.tab_bytes <= kTabBytes), ignored otherwise.
// Chunk sizes the register-copy kernel is compiled for.
bool regcopy_chunk_supported(int64_t chunk_bytes, int vec_bytes);
cudaError_t launch_migrate(const MigrateParams& p, const TabPool& tab, const LaunchCfg& cfg, cudaStream_t stream);
// remp_shared.cu: sharing-preserving ids. first [src_pool], entry_src and excl [num_seqs * max_blocks] are scratch.
cudaError_t launch_dedupe(const int32_t* block_tables, int32_t num_seqs, int32_t max_blocks, int32_t base_block,
                          const int32_t* off, int64_t src_pool, int64_t avail_blocks, int32_t* first,
                          int32_t* entry_src, int32_t* excl, int32_t* dst_block_tables, int4* pairs, int32_t* total,
                          uint32_t* err, cudaStream_t stream, int32_t block_size);

void count_launch(int n = 1);
int64_t launch_count();

// ---- shared host helpers (remp_common.cpp) ----------------------------------------------------
remp_status fail(remp_status st, const std::string& msg);     // records the thread's last error, returns st
remp_status cuda_fail(cudaError_t e, const char* what);
remp_status report_error(remp_status st, const char* msg);
const char* last_error();
remp_status device_pool(int device, cudaMemPool_t* out);      // library-owned memory pool of a device
remp_status trim_pools();
inline size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }

#define REMP_CUDA(call)                                           \
    do {                                                          \
        cudaError_t e_ = (call);                                  \
        if (e_ != cudaSuccess) return remp::cuda_fail(e_, #call); \
    } while (0)

// ---- planner (remp_plan.cpp) ------------------------------------------------------------------
remp_status check_shape(const remp_model_shape& m);

// ---- migration (remp_migrate.cpp) -------------------------------------------------------------
struct ShardView {  // a shard with its strides resolved
    uint64_t base;
    int64_t nb, s_layer, s_kv, s_block, s_head, s_token;
    int64_t extent;  // bytes from base to one past the last byte
};
remp_status ensure_scratch(remp_plan_s* P, int64_t need_pairs, cudaStream_t stream);
void release_scratch(remp_plan_s* P);
remp_status status_from_word(uint32_t w);
// Build the addressing tables of the layers [layer_lo, layer_hi) and launch the migration kernel.
// dst_here (optional, one flag per destination rank): only the flagged ranks are written (the others live on
// other GPUs); planes none of whose replicas is flagged are left out of the launch altogether.
remp_status enqueue_migrate(remp_plan_s* plan, const std::vector<ShardView>& sv, const std::vector<ShardView>& dv,
                            int layer_lo, int layer_hi, cudaStream_t stream,
                            const std::vector<uint8_t>* dst_here = nullptr);

}  // namespace remp

// The opaque plan.
struct remp_plan_s {
    remp_model_shape shape{};
    remp_block_tables tables{};
    remp::TopoMap src, dst;
    std::vector<remp::Item> items;
    std::vector<int32_t> first_item;  // index of the first item of (layer, destination TP rank)

    // derived copy structure
    int run_heads = 0;  // heads per contiguous run = gcd(Hl_src, Hl_dst)
    int n_sub = 0;      // runs per destination block
    int n_groups = 0;   // destination planes: (pp stage, head-owner group, layer, K/V)
    int64_t head_slice_bytes = 0;

    // device scratch owned by the plan: one stream-ordered allocation, carved into the arrays below
    int device = -1;
    int num_sms = 0;
    void* d_block = nullptr;
    cudaStream_t last_stream = nullptr;  // stream of the most recent enqueue; the block is freed on it
    int32_t* d_off = nullptr;    // [num_seqs + 1]
    // status words at the start of the block (kWord* indices): total, error word, preempted count, -, scheduler word
    int32_t* d_total = nullptr;
    uint32_t* d_err = nullptr;
    uint32_t* d_num_preempted = nullptr;  // sequences preempted by the capacity-constrained allocation
    unsigned long long* d_sched = nullptr;  // tile scheduler word of the migration kernels
    long long* d_tile_sums = nullptr;     // [ceil(num_seqs / 1024)] tile sums of the multi-CTA demand scan
    int4* d_pairs = nullptr;     // [pair_cap]
    int64_t pair_cap = 0;
    uint8_t* d_tab = nullptr;     // device copy of the addressing tables when they exceed the kernel parameters
    int64_t tab_cap = 0;          // bytes reserved for it
    std::vector<uint8_t> h_tab;   // the addressing tables of the latest launch
    int32_t h_result[4] = {0, 0, 0, 0};  // read-back of the first four status words

    // state
    bool allocated = false;
    std::vector<int64_t> dst_capacity;
    int32_t base_block = 0;

    // options
    int opt_kernel = 0, opt_ctas_per_sm = 0, opt_vec_bytes = 0, opt_lanes_per_warp = 0, opt_schedule = 0, opt_valid_only = 0, opt_order = 0;
    int opt_alloc_path = 0;  // 0 the library chooses, 1 fused single launch, 2 separate scan and remap launches
    int64_t opt_chunk_bytes = 0, opt_tile_items = 0, opt_wait_spins = 0;
};
