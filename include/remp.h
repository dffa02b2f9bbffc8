/*
 * remp.h - C ABI of the B200 (sm_100a) library for two-dimensional KV-cache migration.
 *
 * The operation is the one section 3.4 of the ReMP paper defines: a paged KV cache sharded for a source
 * topology (TP=a, PP=b) is re-sharded for a destination topology (TP=c, PP=d) so that every logical
 * slice KV[l, b, h] held by rank(l, h, T_old) ends up on rank(l, h, T_new) (section 3.4.1). TP changes
 * split or merge KV-head ranges, PP changes regroup layer ranges, and every sequence's block table is
 * rewritten by a deterministic block remapping (section 3.4.5, "logical block identity preservation").
 * In the basic calls all logical ranks live on one GPU, one allocation per rank, and no peer transfer or
 * collective is used; remp_migrate_kv_exchange covers ranks spread over several GPUs (each GPU pulls what its
 * destination ranks receive), remp_weights_reshard the model weights (section 3.3).
 *
 * Conventions fixed by this library where the paper leaves them open
 *   pp_owner   layers are split into PP contiguous ascending ranges; even split with the first
 *              (L mod PP) stages one layer longer, or explicit boundaries (remp_topo.pp_layer_start).
 *   tp_owner   TP <= H requires TP | H: rank t owns heads [t*H/TP, (t+1)*H/TP).
 *              TP >  H requires H | TP: rep = TP/H consecutive ranks each hold a replica of head t/rep.
 *   rank       rank = pp_rank * TP + tp_rank; all per-rank arrays below are in this order.
 *   replicas   a head replicated on the source side is read from its lowest-numbered owner only.
 *   layout     canonical shard of a rank: [local layer][K,V][block][local head][token][dim], dense.
 *   blocks     whole blocks move (slack tokens of a partial last block included, verbatim).
 *   ids        destination block id of logical block j of sequence s:
 *              base_block + (exclusive prefix sum of ceil(len/block_size) over sequence index)[s] + j,
 *              identical on every destination rank.
 *
 * Threading: a plan may be used by one host thread at a time, and the work of one plan must be ordered on the
 * device (one stream, or streams ordered after one another): its calls share the plan's scratch. Different
 * plans are independent and may run on different streams at once. All device work is enqueued on the stream
 * the caller passes (a cudaStream_t cast to void*; NULL = the legacy default stream) and the calls
 * return without waiting unless stated. For inputs of up to 1024 sequences and 2^18 table entries a switch is two
 * kernel launches - remp_alloc_dst_blocks (with total_blocks = NULL) and remp_migrate_kv - with no memset or copy
 * between them; once the plan's scratch exists (after its first allocation call) the pair can be captured in a
 * CUDA graph and replayed on changed table contents. Errors are returned as statuses; the device code never traps:
 * a condition found on the device is recorded in the plan's error word (see remp_plan_status).
 */
#ifndef REMP_H_
#define REMP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    REMP_OK = 0,
    REMP_ERR_INVALID_ARG = -1,      /* null pointer, negative size, misuse                              */
    REMP_ERR_INVALID_TOPOLOGY = -2, /* TP/PP not legal for the model (see tp_owner / pp_owner above)     */
    REMP_ERR_SHAPE = -3,            /* unsupported shape, stride or alignment                            */
    REMP_ERR_CAPACITY = -4,         /* live blocks do not fit a destination pool (section 3.4.5)         */
    REMP_ERR_ALIAS = -5,            /* a destination shard overlaps a source shard or another destination */
    REMP_ERR_BAD_BLOCK_ID = -6,     /* a live block-table entry is outside the source pool               */
    REMP_ERR_STATE = -7,            /* calls made out of order                                           */
    REMP_ERR_CUDA = -8,             /* a CUDA runtime call failed; remp_last_error() has the text        */
    REMP_ERR_NOMEM = -9,
    REMP_ERR_BAD_LENGTH = -10       /* a sequence length is negative or needs more blocks than a row has */
} remp_status;

/* A topology T = (TP, PP) (section 3.4.1). pp_layer_start: host pointer to PP+1 ascending layer
 * boundaries ([0] = 0, [PP] = num_layers), or NULL for the even split. Read during the call only. */
typedef struct {
    int32_t tp, pp;
    const int32_t* pp_layer_start;
} remp_topo;

/* Model shape. elem_bytes is 1, 2 or 4; elements are opaque bytes (fp8, fp16, bf16 ... are all copied
 * verbatim). block_size*head_dim*elem_bytes must be a multiple of 16. */
typedef struct {
    int32_t num_layers, num_kv_heads, head_dim, block_size, elem_bytes;
} remp_model_shape;

/* The scheduler's frozen KV metadata (section 3.5 "freeze KV metadata"). Both pointers are DEVICE
 * pointers owned by the caller; they must stay valid and unchanged until the work enqueued by
 * remp_alloc_dst_blocks has completed. Row s of block_tables holds ceil(seq_lens[s]/block_size) live
 * source block ids followed by padding (any value; -1 by convention). Length 0 is legal. */
typedef struct {
    int32_t num_seqs, max_blocks_per_seq;
    const int32_t* seq_lens;     /* device, [num_seqs], tokens                      */
    const int32_t* block_tables; /* device, [num_seqs][max_blocks_per_seq], row-major */
} remp_block_tables;

/* One rank's KV pool. base: an address the device can access, 16-byte aligned, owned by the caller: device
 * memory, or page-locked host memory mapped into the device's address space (the kernel then moves the
 * bytes over the host link itself; that is how a swapped-out cache is brought back in a new topology). Strides are in bytes and
 * multiples of 16; 0 selects the canonical dense value ([local layer][K,V][block][local head][token][dim]).
 * stride_layer, stride_kv and stride_block may be anything that keeps slices disjoint. stride_head and
 * stride_token describe the inside of a block and must be the same for all shards of one side: the dense
 * head-major block has stride_head = block_size*head_dim*elem_bytes, stride_token = head_dim*elem_bytes; a
 * token-major block [token][head][dim] has stride_head = head_dim*elem_bytes, stride_token =
 * heads_per_rank*head_dim*elem_bytes (needs head_dim*elem_bytes to be a multiple of 16). Source and
 * destination may differ (the migration then converts). */
typedef struct {
    void* base;
    int64_t num_blocks;
    int64_t stride_layer, stride_kv, stride_block, stride_head, stride_token;
} remp_shard;

typedef struct remp_plan_s remp_plan; /* opaque, owned by the library */

/* What `rank` owns under a topology (section 3.4.1: pp_owner and tp_owner, with the conventions above):
 * out[0], out[1] = its layer range [lo, hi), out[2], out[3] = its KV-head range [lo, hi). Ranks that replicate
 * a head report the same one-head range. out: HOST, 4 x int32. Host work only. */
remp_status remp_rank_ownership(const remp_topo* topo, const remp_model_shape* shape, int32_t rank, int32_t* out);

/* Bytes of the canonical dense shard of `rank` with num_blocks blocks, or a negative remp_status. */
int64_t remp_shard_bytes(const remp_topo* topo, const remp_model_shape* shape, int32_t rank, int64_t num_blocks);

/* Build the migration plan (Algorithm 1): validates both topologies, builds the layer->stage and
 * head->rank maps and the item list (src, dst, layer, head range). Host work only: no CUDA call is made
 * and no device data is read (the plan's small device scratch is created by the first
 * remp_alloc_dst_blocks, on the device current at that time).
 * On success *out is a plan the caller must release with remp_plan_destroy. */
remp_status remp_plan_create(const remp_topo* src, const remp_topo* dst, const remp_model_shape* shape,
                             const remp_block_tables* tables, remp_plan** out);

/* Allocate destination blocks and rewrite the block tables (section 3.4.5: deterministic remapping).
 * Enqueues a prefix scan over per-sequence block demand and the table remapper on `stream`.
 *   dst_capacity_blocks  HOST, [dst.tp*dst.pp]: blocks each destination pool holds
 *   base_block           first destination block id to use (>= 0)
 *   dst_block_tables     DEVICE out, same shape as tables->block_tables (may alias it): ids for live
 *                        entries, -1 elsewhere. Left untouched when the capacity check fails.
 *   total_blocks         HOST out or NULL. Non-NULL makes the call wait for the stream and return
 *                        REMP_ERR_CAPACITY / REMP_ERR_BAD_LENGTH / REMP_ERR_BAD_BLOCK_ID found on the
 *                        device; with NULL those are only recorded (remp_plan_status) and a later
 *                        remp_migrate_kv on the same plan copies nothing when capacity or lengths failed. */
remp_status remp_alloc_dst_blocks(remp_plan* plan, const int64_t* dst_capacity_blocks, int32_t base_block,
                                  int32_t* dst_block_tables, int64_t* total_blocks, void* stream);

/* Capacity-constrained allocation (section 3.4.5 "capacity constraint", section 3.5: when the target
 * provides less KV capacity than the live footprint, selected requests are preempted and their blocks
 * reclaimed). The paper leaves the selection to the scheduler; this call takes the sequences to be in
 * priority order (first come, first served) and preempts the tail: sequence s is KEPT iff the blocks of
 * sequences 0..s together fit below the smallest destination pool (base_block + sum <= capacity). Kept
 * sequences get exactly the ids remp_alloc_dst_blocks would give them; a preempted sequence gets an all -1
 * row and preempted[s] = 1 (0 otherwise), and a following remp_migrate_kv copies no block of it. With enough
 * capacity nothing is preempted and the result equals remp_alloc_dst_blocks. Never returns REMP_ERR_CAPACITY.
 *   preempted      DEVICE out, int32 [num_seqs]
 *   total_blocks   HOST out or NULL: blocks allocated to the kept sequences
 *   num_preempted  HOST out or NULL: sequences preempted (sequences of length 0 behind the cut count too)
 * A non-NULL host output makes the call wait for the stream, as in remp_alloc_dst_blocks. */
remp_status remp_alloc_dst_blocks_preempt(remp_plan* plan, const int64_t* dst_capacity_blocks, int32_t base_block,
                                          int32_t* dst_block_tables, int32_t* preempted, int64_t* total_blocks,
                                          int64_t* num_preempted, void* stream);

/* Sharing-preserving allocation (section 3.4.5 counts shared prefixes among what a switch must leave intact).
 * Live table entries that name the same source block - a prefix held once and used by several sequences -
 * receive the same destination block, so shared prefixes stay shared and are copied once. Distinct source blocks get base_block, base_block+1, ... in the order of their first occurrence
 * when the tables are read row by row; without sharing the result equals remp_alloc_dst_blocks.
 *   src_num_blocks  blocks of the source pools (ids outside [0, src_num_blocks) get a block of their own,
 *                   are never copied and are reported as REMP_ERR_BAD_BLOCK_ID)
 *   total_blocks    HOST out or NULL: DISTINCT blocks allocated (this is what the capacity check uses)
 * A following remp_migrate_kv copies each distinct block once. Scratch of the call (4 bytes per source
 * block and 8 per table entry) comes from the library's pool and is returned in stream order. */
remp_status remp_alloc_dst_blocks_shared(remp_plan* plan, const int64_t* dst_capacity_blocks, int32_t base_block,
                                         int64_t src_num_blocks, int32_t* dst_block_tables, int64_t* total_blocks,
                                         void* stream);

/* Move the cache (sections 3.4.1-3.4.3): for every plan item and live block, copy the head-range slice
 * from the source shard to its place in the destination shard(s); a head the destination replicates is
 * read once and written to every replica. Must follow remp_alloc_dst_blocks (or its _preempt / _shared
 * variant) on the same plan, on the same stream (or one ordered after it). Only enqueues; source shards are never written, so the source
 * topology stays valid if anything fails (section 3.5).
 *   src  HOST array [src.tp*src.pp] of shards, rank order;  dst likewise [dst.tp*dst.pp].
 * dst[r].num_blocks must be >= the capacity given to remp_alloc_dst_blocks for rank r. Destination bytes
 * outside the allocated blocks keep their values. Live entries outside a source pool are skipped and
 * recorded as REMP_ERR_BAD_BLOCK_ID. Returns REMP_ERR_ALIAS if any destination byte range intersects a
 * source byte range or another destination's. */
remp_status remp_migrate_kv(remp_plan* plan, const remp_shard* src, const remp_shard* dst, void* stream);

/* Layer-wise streaming migration (section 3.4.4): move only the layers [layer_lo, layer_hi), so that a caller
 * can allocate the destination storage of a few layers, migrate them, release the source storage of those
 * layers and go on - peak memory is then the cache plus a few layers instead of two caches. Same rules as
 * remp_migrate_kv, except that src[r] / dst[r] describe a buffer that holds ONLY the layers of rank r's stage
 * that fall inside the window, the first of them at `base` (consecutive ones stride_layer apart). Ranks whose
 * stage does not intersect the window are ignored (base may be NULL). Any partition of [0, num_layers) into
 * windows, migrated in any order, gives the result of one remp_migrate_kv. */
remp_status remp_migrate_kv_layers(remp_plan* plan, int32_t layer_lo, int32_t layer_hi, const remp_shard* src,
                                   const remp_shard* dst, void* stream);

/* ---- logical ranks spread over several GPUs ----
 *
 * Section 3.4.2 defines the plan from the receiver's side and notes that the send side is its mirror image;
 * section 3.4.3 executes an item as a local copy when source and destination rank share a device and as a remote
 * transfer otherwise. Here every GPU (one process each) holds the shards of the ranks mapped to it and PULLS what its
 * own destination ranks receive: local items are local copies, remote items are plain loads from the owner's memory
 * over NVLink (memory the caller has made addressable from this device: peer access inside one process, an IPC or
 * symmetric-memory mapping between processes). Nothing is pushed, so no GPU waits for another inside the kernel;
 * the caller orders "sources are final" before and "all pulls are done" after with its own barrier.
 *
 * remp_plan_partition: the items of the plan seen from `device`. Rows of 6 int32:
 *   recv_items  (src rank, dst rank, layer, head_lo, head_hi, device of the src rank) for every item whose
 *               destination rank is on `device` - local ones (6th column == device) and remote ones alike;
 *   send_items  (src rank, dst rank, layer, head_lo, head_hi, device of the dst rank) for every item whose source
 *               rank is on `device` and whose destination rank is on another device: the mirror image of that
 *               device's remote recv items.
 *   src_rank_device / dst_rank_device  HOST, [src ranks] / [dst ranks]: device index of every rank (any ints >= 0)
 *   recv_items / send_items            HOST out or NULL (NULL: only the counts are returned)
 * Host work only. */
remp_status remp_plan_partition(const remp_plan* plan, const int32_t* src_rank_device, const int32_t* dst_rank_device,
                                int32_t device, int32_t* recv_items, int32_t* num_recv, int32_t* send_items,
                                int32_t* num_send);

/* remp_migrate_kv for the destination ranks mapped to `device` only (the GPU current in this process): every recv
 * item of remp_plan_partition(plan, ..., device) is executed, every other item is left to the device that owns
 * its destination rank. The calls of all devices together give the result of one remp_migrate_kv. Each process
 * makes its own plan from its own copy of the tables and runs remp_alloc_dst_blocks itself first: the ids are
 * deterministic, so every device computes the same tables.
 *   src   HOST [src ranks]: base = an address THIS device can load from (local or peer memory); entries of source
 *         ranks this device receives nothing from are ignored (base may be NULL)
 *   dst   HOST [dst ranks]: entries of ranks on other devices are ignored
 * Remote sources are read with ordinary loads by the register-copy and strided-row kernels; the bulk-copy kernel
 * (REMP_OPT_KERNEL = 2) is refused with REMP_ERR_INVALID_ARG when any needed source rank is on another device.
 * Otherwise as remp_migrate_kv (only enqueues; source shards are never written). */
remp_status remp_migrate_kv_exchange(remp_plan* plan, const int32_t* src_rank_device, const int32_t* dst_rank_device,
                                     int32_t device, const remp_shard* src, const remp_shard* dst, void* stream);

/* Wait for `stream` and translate the plan's device error word into a status (REMP_OK if clear). */
remp_status remp_plan_status(remp_plan* plan, void* stream);

/* Release a plan. Work already enqueued with it may still be in flight: the plan's device scratch is
 * freed in stream order on the stream the plan was last used with, which must still exist. */
void remp_plan_destroy(remp_plan* plan);

/* Message of the last failing call on this thread (never NULL). */
const char* remp_last_error(void);

/* ---- host-resident caches ----
 *
 * The same re-sharding (sections 3.4.1-3.4.3) for a cache that lives in HOST memory (a swapped-out or
 * sleeping instance), done in one synchronous call: tables go to the device, destination blocks are
 * allocated as in remp_alloc_dst_blocks, then the cache moves in one of two ways.
 *   direct   (window_layers = 0 and every shard buffer is page-locked memory mapped into the device's
 *            address space, e.g. cudaHostAlloc / cudaHostRegister): the migration kernel reads the source
 *            shards and writes the destination shards in host memory itself, one launch, no staging; only
 *            live blocks cross the link.
 *   staged   (otherwise): the layers stream through two device staging slots in windows so that
 *            host->device copies, the migration kernel and device->host copies of consecutive windows
 *            overlap (the layer-wise streaming of section 3.4.4); device memory used: two windows of source
 *            and destination layers from the library's pool. Pageable buffers work but copy synchronously.
 *   seq_lens, block_tables   HOST in;  dst_block_tables HOST out (same shape), total_blocks HOST out
 *   src_shards / dst_shards  HOST arrays in rank order; each base is HOST memory holding the canonical
 *                            dense shard ([local layer][K,V][block][local head][token][dim])
 *   window_layers            0: the library chooses (direct if possible and the source pools hold more than a
 *                            few percent of unused blocks, else staged windows of about 1 GiB of source);
 *                            > 0: staged with this many layers per window
 *   h2d_bytes, d2h_bytes     HOST out or NULL: bytes that crossed the link in each direction
 * Only the allocated block range [base_block, base_block+total) of every destination (layer, K/V) plane
 * is written; all other destination bytes keep their values. Source buffers are only read.
 * Returns when the destination is complete; errors as for remp_alloc_dst_blocks / remp_migrate_kv (REMP_ERR_ALIAS,
 * checked before anything moves, when a destination buffer overlaps a source buffer or another destination buffer). */
typedef struct {
    void* base;
    int64_t num_blocks;
} remp_host_shard;
remp_status remp_reshard_host(const remp_topo* src, const remp_topo* dst, const remp_model_shape* shape,
                              int32_t num_seqs, int32_t max_blocks_per_seq, const int32_t* seq_lens,
                              const int32_t* block_tables, const remp_host_shard* src_shards,
                              const remp_host_shard* dst_shards, int32_t base_block, int32_t window_layers,
                              int32_t* dst_block_tables, int64_t* total_blocks, int64_t* h2d_bytes,
                              int64_t* d2h_bytes);

/* ---- model weights from a host store (section 3.3, "Shared Model Weight Store") ----
 *
 * The paper keeps the full model state once in host memory and lets every worker rebuild its GPU shard for the
 * target topology from it: PP selects the layer range, TP slices the partitioned parameters, replicated parameters
 * are taken whole. This is that materialisation for all target ranks (one device allocation per rank, as for the
 * KV cache), with the same stage map (pp_owner) as the KV path.
 *
 * The store is a list of parameter descriptions. Every tensor is a row-major [rows][cols] array in HOST memory.
 *   partition  REMP_W_REPLICATED        every TP rank takes the whole tensor
 *              REMP_W_SPLIT_ROWS        rows split evenly across TP (column-parallel linear layers, vocabulary-
 *                                       parallel embeddings): rank t takes rows [t*rows/TP, (t+1)*rows/TP)
 *              REMP_W_SPLIT_COLS        columns split evenly across TP (row-parallel linear layers)
 *              REMP_W_SPLIT_ROW_GROUPS  rows form `groups` equal groups (the KV heads of a K/V projection); groups
 *                                       are dealt to TP ranks exactly as KV heads are (tp_owner above): TP <= groups
 *                                       needs TP | groups, TP > groups needs groups | TP and replicates
 *   scope      REMP_W_EVERY_LAYER       one instance per layer, layer l at host_base + l*layer_stride; a rank gets
 *                                       the instances of the layers of its stage
 *              REMP_W_FIRST_STAGE       one instance, only ranks of stage 0 get it (embeddings)
 *              REMP_W_LAST_STAGE        one instance, only ranks of the last stage get it (final norm, output head)
 * A rank's shard is packed by the library: first-stage parameters, then for each layer of the stage the per-layer
 * parameters in list order, then last-stage parameters; every slice is dense row-major [local rows][local cols]
 * and starts on a 256-byte boundary (remp_weight_slice tells where). A slice's row (local cols * elem_bytes) and
 * its column offset in bytes must be multiples of 16, host_base and layer_stride too, else REMP_ERR_SHAPE. */
typedef enum { REMP_W_REPLICATED = 0, REMP_W_SPLIT_ROWS = 1, REMP_W_SPLIT_COLS = 2, REMP_W_SPLIT_ROW_GROUPS = 3 } remp_weight_partition;
typedef enum { REMP_W_EVERY_LAYER = 0, REMP_W_FIRST_STAGE = 1, REMP_W_LAST_STAGE = 2 } remp_weight_scope;
typedef struct {
    const void* host_base;
    int64_t layer_stride; /* bytes; REMP_W_EVERY_LAYER only */
    int64_t rows, cols;   /* full extent in elements */
    int32_t elem_bytes;   /* 1, 2 or 4 */
    int32_t partition;    /* remp_weight_partition */
    int32_t groups;       /* REMP_W_SPLIT_ROW_GROUPS only */
    int32_t scope;        /* remp_weight_scope */
} remp_weight_param;

/* Bytes of `rank`'s packed shard under `topo`, or a negative remp_status. Host work only. */
int64_t remp_weight_shard_bytes(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                                int32_t num_params, int32_t rank);

/* Where parameter `param` (of global layer `layer`; ignored for the other scopes) sits in `rank`'s shard and its
 * local extent. REMP_ERR_INVALID_ARG when the rank does not hold it. All outputs HOST. Host work only. */
remp_status remp_weight_slice(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                              int32_t num_params, int32_t rank, int32_t param, int32_t layer, int64_t* offset,
                              int64_t* rows, int64_t* cols);

/* Materialise the shards of all ranks of `topo` from the host store.
 *   dst_shards  HOST array [topo.tp*topo.pp] of DEVICE pointers, each remp_weight_shard_bytes long, 256-byte aligned
 *   h2d_bytes   HOST out or NULL: bytes that crossed the host link
 * When every tensor of the store is page-locked memory mapped into the device's address space, one gather kernel
 * reads the slices straight out of host memory (only enqueues on `stream`; the store must stay unchanged until
 * that work is done). Otherwise every slice is one strided copy on the copy engine (pageable memory makes those
 * copies synchronous). Padding bytes between slices keep their values.
 *   max_ctas    0: the gather kernel fills the GPU (fastest when nothing else runs). > 0: at most that many thread
 *               blocks, so that a KV migration enqueued on another stream runs beside the weight load instead of
 *               behind it (the overlap of model reload and cache migration of section 3.4.4): the host link needs few
 *               bytes in flight - a quarter of the SM count keeps 98 % of its rate - while a grid that fills the
 *               GPU holds every SM until the load is done. Ignored on the copy-engine path. < 0: REMP_ERR_INVALID_ARG. */
remp_status remp_weights_reshard(const remp_topo* topo, int32_t num_layers, const remp_weight_param* params,
                                 int32_t num_params, void* const* dst_shards, int64_t* h2d_bytes, int32_t max_ctas,
                                 void* stream);

/* ---- introspection (tests, benchmarks) ---- */

/* Number of Algorithm-1 items, and the items themselves as rows of 5 int32:
 * (src rank, dst rank, layer, head_lo, head_hi). out: HOST, [num_items][5]. The source rank of an item whose heads
 * the source topology replicates is always the lowest-numbered owner, so no replica column is needed. */
int32_t remp_plan_num_items(const remp_plan* plan);
remp_status remp_plan_get_items(const remp_plan* plan, int32_t* out);

/* Algorithmic traffic of one migration of total_blocks live blocks: bytes read (each distinct source
 * byte once) and bytes written (times the destination replication). */
remp_status remp_plan_traffic(const remp_plan* plan, int64_t total_blocks, int64_t* bytes_read, int64_t* bytes_written);

/* Same, counted in tokens: traffic of a migration in valid-tokens-only mode that moves valid_tokens tokens. */
remp_status remp_plan_traffic_tokens(const remp_plan* plan, int64_t valid_tokens, int64_t* bytes_read,
                                     int64_t* bytes_written);

/* Tuning knobs; value 0 restores the default. Unknown keys return REMP_ERR_INVALID_ARG. */
typedef enum {
    REMP_OPT_KERNEL = 1,       /* 1 = register copy (16-byte loads/stores), 2 = bulk-copy ring through shared memory */
    REMP_OPT_CTAS_PER_SM = 2,  /* persistent CTAs per SM */
    REMP_OPT_CHUNK_BYTES = 3,  /* bytes one warp (kernel 1: 512, 1024, 2048, 4096 or 8192) or one ring stage (kernel 2: any
                                  multiple of 512 up to 32768) moves at a time; a value the selected kernel does not
                                  take makes remp_migrate_kv return REMP_ERR_INVALID_ARG before anything is enqueued */
    REMP_OPT_VEC_BYTES = 4,    /* kernel 1: bytes per load/store instruction, 16 or 32 */
    REMP_OPT_TILE_ITEMS = 5,   /* kernel 1: consecutive chunks a CTA takes before striding by the grid */
    REMP_OPT_LANES_PER_WARP = 6, /* kernel 2: stage-owning lanes per warp */
    REMP_OPT_SCHEDULE = 7,     /* kernel 1: 1 = tiles assigned round-robin; 2 = CTAs draw tiles from a device counter
                                  (default); 3 = every warp draws its own tiles */
    REMP_OPT_VALID_TOKENS_ONLY = 8, /* 1: of a partial last block copy only the tokens in use (tokens
                                  j*block_size .. len-1); the slack token slots of the destination block keep their
                                  bytes. Default 0: whole blocks move. Not combined with shared-prefix allocation
                                  (shared blocks always move whole). */
    REMP_OPT_ORDER = 9,        /* order of the work: 2 = one destination rank's (layer, K/V) plane after the other;
                                  1 = per (layer, K/V) all destination ranks together, block by block; 0 = the
                                  library chooses (1 when the pieces a block gives to different destination ranks share
                                  memory lines: head slices or rows below 128 bytes, or strided rows below 1 KiB that
                                  are not a power of two, cut out of wider source rows) */
    REMP_OPT_ALLOC_PATH = 10,  /* remp_alloc_dst_blocks and its _preempt variant: 1 = one fused launch (prefix scan,
                                  table rewrite and status words in a single thread-block cluster; at most 1024
                                  sequences and 2^18 table entries, else REMP_ERR_INVALID_ARG), 2 = separate scan and
                                  remap launches, 0 = the library chooses (fused whenever the input is in its range).
                                  Both give identical results. */
    REMP_OPT_WAIT_SPINS = 11   /* kernel 2, a test aid: value v > 0 lets a copy barrier be polled v-1 times before it is
                                  given up and reported as REMP_ERR_CUDA (0 = the built-in limit of 2^20 polls). A given-up
                                  item keeps its destination bytes; every other item is copied as usual. */
} remp_option;
remp_status remp_plan_set_option(remp_plan* plan, int32_t key, int64_t value);

/* The library keeps the scratch of destroyed plans in a per-device memory pool so that the next switch costs no
 * device allocation. This call hands unused pool memory back to the driver (memory of live plans and of work
 * still in flight is not touched). */
remp_status remp_release_cached_memory(void);

/* Kernels launched by this library in this process so far. */
int64_t remp_kernel_launch_count(void);

/* ---- for callers that cannot allocate device memory ----
 *
 * (The paper has no counterpart: this is a packaging variant of remp_alloc_dst_blocks' table rewrite.)
 * Some hosts of this library may not call cudaMalloc at the time a topology switch happens: a serving
 * process that handed all free HBM to its KV pools at start-up, code running between the iterations of a
 * latency-critical decode loop where an allocation would stall on the driver, or an embedder whose
 * memory budget is fixed by an outer framework. remp_remap_tables_noalloc gives them the destination block
 * ids and the rewritten tables without any allocation: the prefix offsets, the block total and the status
 * word it needs between its two kernels live in a fixed array of (REMP_NOALLOC_MAX_SEQS + 4) int32
 * (256 KiB) inside the library image, which every GPU that loads the library holds until the process exits.
 *
 *   seq_lens           DEVICE in,  [num_seqs] tokens
 *   capacity_blocks    blocks the smallest destination pool holds; ids base_block .. base_block+total-1
 *                      must fit below it
 *   dst_block_tables   DEVICE out, [num_seqs][max_blocks_per_seq]: base_block + prefix + j for the
 *                      ceil(len/block_size) live entries of a row, -1 for its padding (the same values
 *                      remp_alloc_dst_blocks writes). Untouched when the status word reports a capacity,
 *                      length or overflow error.
 *   result             DEVICE out, 2 x int32: [0] total blocks, [1] status word (0 = ok; bit 0 capacity
 *                      exceeded, bit 1 bad length, bit 2 total does not fit 32 bits). The caller reads it
 *                      back when and how it likes; the call itself never waits.
 * num_seqs above REMP_NOALLOC_MAX_SEQS is rejected with REMP_ERR_INVALID_ARG before anything is enqueued.
 * The call makes no cudaMalloc/cudaFree and uses no allocating routine; it enqueues one memset and two
 * kernels on `stream`. The first call on each device also looks up the array's device address (with that
 * device current); make that first call outside any stream capture. All calls on a device share the one
 * array, which still holds the previous call's contents (the words that must start at zero are cleared by
 * the call itself): two calls whose kernels may overlap on the GPU - different streams without an ordering
 * between them, or several host threads - race on it and must be serialised by the caller. */
#define REMP_NOALLOC_MAX_SEQS 65536
remp_status remp_remap_tables_noalloc(const int32_t* seq_lens, int32_t num_seqs, int32_t max_blocks_per_seq,
                                      int32_t block_size, int32_t base_block, int64_t capacity_blocks,
                                      int32_t* dst_block_tables, int32_t* result, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* REMP_H_ */
