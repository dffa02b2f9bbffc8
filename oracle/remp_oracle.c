/*
 * CPU oracle for two-dimensional KV-cache migration (paper section 3.4).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition the CUDA library is checked against.
 * It shares no code, header, table or helper with the CUDA path and must never be called from it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * What it computes (section 3.4.1, the preservation law KV[l,b,h] on rank(l,h,T_old) -> KV[l,b,h] on
 * rank(l,h,T_new)), with the readings the paper leaves open fixed as follows:
 *   - pp_owner: contiguous ascending layer ranges; even split, the first (L mod PP) stages one layer
 *     longer; or explicit boundaries.
 *   - tp_owner / head_range: TP <= H needs TP | H, rank t owns heads [t*H/TP, (t+1)*H/TP);
 *     TP > H needs H | TP, rep = TP/H consecutive ranks all own the single head t/rep (replication is
 *     the exception the head-coverage invariant of section 3.4.5 allows).
 *   - rank(pp, tp) = pp*TP + tp.
 *   - a replicated source head is read from its lowest-numbered owner.
 *   - shard layout of rank (p,t): [local layer][K,V][block][local head][token][dim], dense.
 *   - destination block ids: base + exclusive running sum of ceil(len/bs) in sequence order + j, the
 *     same on every destination rank (the deterministic block remapping of section 3.4.5); whole
 *     blocks move, slack tokens of a partial block included; every other destination byte is kept.
 *
 * Pins (see tests, CPU-only): exactly-once coverage counted by an independent source-driven enumerator,
 * closed-form plan sizes of Algorithm 1, reductions to numpy slicing/concatenation/fancy indexing,
 * round trips, and brute force on tiny inputs. The paper prints no worked example, so parity with the
 * paper's own figures is unpinned; the definition itself is pinned by the above.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t tp, pp;
    const int32_t* layer_start; /* NULL = even split; else pp+1 ascending boundaries, [0]=0, [pp]=L */
} orc_topo;

typedef struct {
    int32_t L, H, D, bs, e;
} orc_shape;

/* ------------------------------------------------------------------------------------------------
 * Ownership functions (section 3.4.1: pp_owner, tp_owner, rank)
 * ---------------------------------------------------------------------------------------------- */

/* First layer of stage p; p == PP gives L. */
int orc_stage_first(const orc_topo* T, int L, int p) {
    if (T->layer_start) return T->layer_start[p];
    int q = L / T->pp, r = L % T->pp;
    int first = 0;
    for (int i = 0; i < p; ++i) first += q + (i < r ? 1 : 0);
    return first;
}

int orc_pp_owner(const orc_topo* T, int L, int l) {
    for (int p = 0; p < T->pp; ++p)
        if (l >= orc_stage_first(T, L, p) && l < orc_stage_first(T, L, p + 1)) return p;
    return -1;
}

int orc_rep(const orc_topo* T, int H) { return T->tp > H ? T->tp / H : 1; }
int orc_heads_per_rank(const orc_topo* T, int H) { return T->tp > H ? 1 : H / T->tp; }

/* head_range(t, TP, H) of Algorithm 1: [lo, hi). */
int orc_head_lo(const orc_topo* T, int H, int t) {
    return T->tp > H ? t / (T->tp / H) : t * (H / T->tp);
}
int orc_head_hi(const orc_topo* T, int H, int t) { return orc_head_lo(T, H, t) + orc_heads_per_rank(T, H); }

int orc_owns_head(const orc_topo* T, int H, int t, int h) {
    return h >= orc_head_lo(T, H, t) && h < orc_head_hi(T, H, t);
}

/* tp_owner(h, TP): the lowest TP rank that owns head h. */
int orc_tp_owner(const orc_topo* T, int H, int h) {
    for (int t = 0; t < T->tp; ++t)
        if (orc_owns_head(T, H, t, h)) return t;
    return -1;
}

int orc_rank(const orc_topo* T, int p, int t) { return p * T->tp + t; }

/* 0 when the topology is legal for the model. */
int orc_topo_check(const orc_topo* T, const orc_shape* m) {
    if (T->tp < 1 || T->pp < 1 || m->L < 1 || m->H < 1) return 1;
    if (T->pp > m->L) return 2;
    if (T->tp <= m->H ? (m->H % T->tp != 0) : (T->tp % m->H != 0)) return 3;
    if (T->layer_start) {
        if (T->layer_start[0] != 0 || T->layer_start[T->pp] != m->L) return 4;
        for (int p = 0; p < T->pp; ++p)
            if (T->layer_start[p + 1] <= T->layer_start[p]) return 4;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Shard layout: [local layer][2][block][local head][token][dim]
 * ---------------------------------------------------------------------------------------------- */

int64_t orc_head_slice_bytes(const orc_shape* m) { return (int64_t)m->bs * m->D * m->e; }

int64_t orc_layer_slab_bytes(const orc_topo* T, const orc_shape* m, int64_t nb) {
    return 2 * nb * orc_heads_per_rank(T, m->H) * orc_head_slice_bytes(m);
}

int64_t orc_shard_bytes(const orc_topo* T, const orc_shape* m, int rank, int64_t nb) {
    int p = rank / T->tp;
    int nl = orc_stage_first(T, m->L, p + 1) - orc_stage_first(T, m->L, p);
    return nl * orc_layer_slab_bytes(T, m, nb);
}

/* Byte offset inside a layer slab of TP rank t of element (kv, blk, global head h, tok, dim).
 * layout 0: [K,V][block][local head][token][dim] (head-major, the canonical layout);
 * layout 1: [K,V][block][token][local head][dim] (token-major blocks, as attention kernels often keep them). */
static int64_t slab_offset_l(const orc_topo* T, const orc_shape* m, int64_t nb, int t, int kv, int64_t blk, int h,
                             int tok, int dim, int layout) {
    int hl = orc_heads_per_rank(T, m->H);
    int hloc = h - orc_head_lo(T, m->H, t);
    if (layout == 1) return ((((kv * nb + blk) * m->bs + tok) * hl + hloc) * (int64_t)m->D + dim) * m->e;
    return ((((kv * nb + blk) * hl + hloc) * m->bs + tok) * (int64_t)m->D + dim) * m->e;
}

static int64_t slab_offset(const orc_topo* T, const orc_shape* m, int64_t nb, int t, int kv, int64_t blk, int h,
                           int tok, int dim) {
    return slab_offset_l(T, m, nb, t, kv, blk, h, tok, dim, 0);
}

/* Byte offset inside the shard of `rank`, or -1 if that rank does not own (layer l, head h). */
int64_t orc_offset(const orc_topo* T, const orc_shape* m, int rank, int64_t nb, int l, int kv, int64_t blk, int h,
                   int tok, int dim) {
    int p = rank / T->tp, t = rank % T->tp;
    if (orc_pp_owner(T, m->L, l) != p || !orc_owns_head(T, m->H, t, h)) return -1;
    int lloc = l - orc_stage_first(T, m->L, p);
    return lloc * orc_layer_slab_bytes(T, m, nb) + slab_offset(T, m, nb, t, kv, blk, h, tok, dim);
}

/* ------------------------------------------------------------------------------------------------
 * Destination block allocation: serial running sum (deterministic remapping, section 3.4.5)
 * ---------------------------------------------------------------------------------------------- */

/* Returns the number of blocks allocated; -1 if base+total exceeds a destination capacity (nothing is
 * written then); -2 if a sequence needs more entries than the table is wide. off (n_seq+1) may be NULL. */
int64_t orc_alloc(int n_seq, int maxb, const int32_t* lens, int bs, int32_t base, const int64_t* caps, int nranks,
                  int32_t* dst_bt, int32_t* off) {
    int64_t run = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        if (lens[s] < 0 || need > maxb) return -2;
        run += need;
    }
    for (int r = 0; r < nranks; ++r)
        if (base + run > caps[r]) return -1;
    run = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        if (off) off[s] = (int32_t)run;
        for (int j = 0; j < maxb; ++j) dst_bt[(int64_t)s * maxb + j] = j < need ? (int32_t)(base + run + j) : -1;
        run += need;
    }
    if (off) off[n_seq] = (int32_t)run;
    return run;
}

/* Capacity-constrained allocation (section 3.4.5, "capacity constraint": when the target holds less than
 * the live footprint, selected requests are preempted and their blocks reclaimed). The paper leaves the
 * selection open; the reading here follows first-come-first-served serving: sequences are in priority
 * order, the tail is preempted - sequence s is kept iff the blocks of sequences 0..s together fit below the
 * smallest destination pool. Kept sequences get ids exactly as in orc_alloc; preempted ones get an all -1
 * row and preempted[s] = 1. Returns the number of blocks of the kept sequences, or -2 on a bad length. */
int64_t orc_alloc_preempt(int n_seq, int maxb, const int32_t* lens, int bs, int32_t base, const int64_t* caps,
                          int nranks, int32_t* dst_bt, int32_t* preempted) {
    int64_t avail = INT64_MAX;
    for (int r = 0; r < nranks; ++r)
        if (caps[r] - base < avail) avail = caps[r] - base;
    if (avail < 0) avail = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        if (lens[s] < 0 || need > maxb) return -2;
    }
    int64_t run = 0;
    int cut = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        if (!cut && run + need > avail) cut = 1;
        preempted[s] = cut;
        for (int j = 0; j < maxb; ++j)
            dst_bt[(int64_t)s * maxb + j] = (!cut && j < need) ? (int32_t)(base + run + j) : -1;
        if (!cut) run += need;
    }
    return run;
}

/* Sharing-preserving allocation (section 3.4.5 lists prefixes among the things whose cache contents a switch
 * must not disturb). Live table entries that name the same source block - a prefix held once and used by
 * several sequences - receive the same destination block; distinct source blocks receive distinct
 * ids base, base+1, ... in the order of their first occurrence when the tables are read row by row.
 * src_pool: number of blocks of the source pools; an entry outside [0, src_pool) is given a block of its own
 * and reported (return value's sign is not used for it: *bad is set).
 * Returns the number of blocks allocated, -1 when they exceed a destination capacity (nothing written),
 * -2 on a bad length. */
int64_t orc_alloc_shared(int n_seq, int maxb, const int32_t* lens, const int32_t* bt, int bs, int32_t base,
                         int64_t src_pool, const int64_t* caps, int nranks, int32_t* dst_bt, int32_t* bad) {
    int64_t entries = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        if (lens[s] < 0 || need > maxb) return -2;
        entries += need;
    }
    int32_t* seen = (int32_t*)malloc(sizeof(int32_t) * (size_t)(src_pool > 0 ? src_pool : 1));
    int32_t* out = (int32_t*)malloc(sizeof(int32_t) * (size_t)(entries > 0 ? entries : 1));
    for (int64_t b = 0; b < src_pool; ++b) seen[b] = -1;
    int64_t next = 0, k = 0;
    *bad = 0;
    for (int s = 0; s < n_seq; ++s) {
        int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
        for (int64_t j = 0; j < need; ++j, ++k) {
            int64_t sb = bt[(int64_t)s * maxb + j];
            if (sb < 0 || sb >= src_pool) {
                *bad = 1;
                out[k] = (int32_t)(base + next++);
            } else {
                if (seen[sb] < 0) seen[sb] = (int32_t)(base + next++);
                out[k] = seen[sb];
            }
        }
    }
    int fits = 1;
    for (int r = 0; r < nranks; ++r)
        if (base + next > caps[r]) fits = 0;
    if (fits) {
        k = 0;
        for (int s = 0; s < n_seq; ++s) {
            int64_t need = ((int64_t)lens[s] + bs - 1) / bs;
            for (int j = 0; j < maxb; ++j) dst_bt[(int64_t)s * maxb + j] = j < need ? out[k++] : -1;
        }
    }
    free(seen);
    free(out);
    return fits ? next : -1;
}

/* ------------------------------------------------------------------------------------------------
 * Migration plan (what Algorithm 1 produces), written from the ownership definition of section 3.4.1 rather
 * than as interval arithmetic: for every layer and every destination TP rank, walk the KV heads in ascending
 * order; a head the rank owns has to arrive from whoever holds it on the source side. Consecutive heads with
 * the same single sender form one item. One row per item: (src rank, dst rank, layer, h_lo, h_hi).
 * A head that the source side replicates has several holders: with dedupe != 0 only the lowest-numbered one
 * sends it; with dedupe == 0 every holder does (one item each), which is what the algorithm yields when it
 * is applied as printed to a replicated source.
 * Returns the number of items (rows beyond cap are counted but not written).
 * ---------------------------------------------------------------------------------------------- */
static void plan_emit(int32_t* items, int cap, int* n, int src_rank, int dst_rank, int layer, int h_lo, int h_hi) {
    if (*n < cap) {
        int32_t* it = items + 5 * (int64_t)*n;
        it[0] = src_rank;
        it[1] = dst_rank;
        it[2] = layer;
        it[3] = h_lo;
        it[4] = h_hi;
    }
    ++*n;
}

int orc_plan(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int dedupe, int32_t* items, int cap) {
    int n = 0;
    for (int layer = 0; layer < m->L; ++layer) {
        const int src_stage = orc_pp_owner(S, m->L, layer);
        const int dst_stage = orc_pp_owner(Dt, m->L, layer);
        for (int td = 0; td < Dt->tp; ++td) {
            const int dst_rank = orc_rank(Dt, dst_stage, td);
            int sender = -1, first_head = 0; /* open item: heads [first_head, h) all come from TP rank `sender` */
            for (int h = 0; h <= m->H; ++h) {
                const int wanted = h < m->H && orc_owns_head(Dt, m->H, td, h);
                int holders = 0, lowest = -1;
                if (wanted)
                    for (int ts = S->tp - 1; ts >= 0; --ts)
                        if (orc_owns_head(S, m->H, ts, h)) {
                            ++holders;
                            lowest = ts;
                        }
                const int single = wanted && (dedupe || holders == 1);
                if (sender >= 0 && !(single && lowest == sender)) { /* the open item ends before head h */
                    plan_emit(items, cap, &n, orc_rank(S, src_stage, sender), dst_rank, layer, first_head, h);
                    sender = -1;
                }
                if (!wanted) continue;
                if (single) {
                    if (sender < 0) {
                        sender = lowest;
                        first_head = h;
                    }
                } else { /* every holder of a replicated head sends it */
                    for (int ts = 0; ts < S->tp; ++ts)
                        if (orc_owns_head(S, m->H, ts, h))
                            plan_emit(items, cap, &n, orc_rank(S, src_stage, ts), dst_rank, layer, h, h + 1);
                }
            }
        }
    }
    return n;
}

/* ------------------------------------------------------------------------------------------------
 * Migration of one layer, from the layer slabs of the source TP ranks of the stage that owns it to the
 * layer slabs of the destination TP ranks [t_lo, t_hi) of the stage that will own it.
 * mode 0: one element (e bytes) at a time; mode 1: one (token) row of D*e bytes at a time.
 * Returns 0, or -6 on a source/destination block id outside its pool (that block is skipped).
 * ---------------------------------------------------------------------------------------------- */
/* valid_only != 0: of a partial last block only the tokens the sequence has written are copied
 * (tokens j*bs .. len-1); the slack token slots of the destination block keep their bytes. */
int orc_migrate_layer_ex(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb,
                         const int32_t* lens, const int32_t* bt, const int32_t* dst_bt,
                         const uint8_t* const* src_slab, const int64_t* src_nb, uint8_t* const* dst_slab,
                         const int64_t* dst_nb, int t_lo, int t_hi, int mode, int src_layout, int dst_layout,
                         int valid_only) {
    int rc = 0;
    for (int t2 = t_lo; t2 < t_hi; ++t2) {
        for (int kv = 0; kv < 2; ++kv) {
            for (int s = 0; s < n_seq; ++s) {
                int64_t need = ((int64_t)lens[s] + m->bs - 1) / m->bs;
                for (int64_t j = 0; j < need; ++j) {
                    int64_t sb = bt[(int64_t)s * maxb + j];
                    int64_t db = dst_bt[(int64_t)s * maxb + j];
                    for (int h = 0; h < m->H; ++h) {
                        if (!orc_owns_head(Dt, m->H, t2, h)) continue;
                        int t1 = orc_tp_owner(S, m->H, h);
                        if (sb < 0 || sb >= src_nb[t1] || db < 0 || db >= dst_nb[t2]) {
                            rc = -6;
                            continue;
                        }
                        int64_t ntok = m->bs;
                        if (valid_only && lens[s] - j * m->bs < ntok) ntok = lens[s] - j * m->bs;
                        for (int tok = 0; tok < ntok; ++tok) {
                            if (mode == 1) {
                                memcpy(dst_slab[t2] + slab_offset_l(Dt, m, dst_nb[t2], t2, kv, db, h, tok, 0, dst_layout),
                                       src_slab[t1] + slab_offset_l(S, m, src_nb[t1], t1, kv, sb, h, tok, 0, src_layout),
                                       (size_t)m->D * m->e);
                            } else {
                                for (int d = 0; d < m->D; ++d) {
                                    const uint8_t* a =
                                        src_slab[t1] + slab_offset_l(S, m, src_nb[t1], t1, kv, sb, h, tok, d, src_layout);
                                    uint8_t* b =
                                        dst_slab[t2] + slab_offset_l(Dt, m, dst_nb[t2], t2, kv, db, h, tok, d, dst_layout);
                                    for (int q = 0; q < m->e; ++q) b[q] = a[q];
                                }
                            }
                        }
                    }
                }
            }
        }
    }
    return rc;
}

int orc_migrate_layer_layout(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb,
                             const int32_t* lens, const int32_t* bt, const int32_t* dst_bt,
                             const uint8_t* const* src_slab, const int64_t* src_nb, uint8_t* const* dst_slab,
                             const int64_t* dst_nb, int t_lo, int t_hi, int mode, int src_layout, int dst_layout) {
    return orc_migrate_layer_ex(S, Dt, m, n_seq, maxb, lens, bt, dst_bt, src_slab, src_nb, dst_slab, dst_nb, t_lo, t_hi,
                                mode, src_layout, dst_layout, 0);
}

int orc_migrate_layer(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb,
                      const int32_t* lens, const int32_t* bt, const int32_t* dst_bt, const uint8_t* const* src_slab,
                      const int64_t* src_nb, uint8_t* const* dst_slab, const int64_t* dst_nb, int t_lo, int t_hi,
                      int mode) {
    return orc_migrate_layer_layout(S, Dt, m, n_seq, maxb, lens, bt, dst_bt, src_slab, src_nb, dst_slab, dst_nb, t_lo,
                                    t_hi, mode, 0, 0);
}

/* ------------------------------------------------------------------------------------------------
 * Whole-cache migration over layers [layer_lo, layer_hi): src[r] / dst[r] are shard base pointers in
 * rank order, src_nb / dst_nb the pool sizes per rank. nthreads > 1 splits the (layer, destination TP
 * rank) tasks over threads (each destination byte has one writer, so tasks are independent).
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    const orc_topo *S, *Dt;
    const orc_shape* m;
    int n_seq, maxb;
    const int32_t *lens, *bt, *dst_bt;
    const uint8_t* const* src;
    const int64_t* src_nb;
    uint8_t* const* dst;
    const int64_t* dst_nb;
    int mode, layer_lo, layer_hi;
    int src_layout, dst_layout, valid_only;
    int next_task; /* guarded by mu */
    int rc;
    pthread_mutex_t mu;
} job_t;

static int run_task(job_t* J, int task) {
    const orc_topo *S = J->S, *Dt = J->Dt;
    const orc_shape* m = J->m;
    int l = J->layer_lo + task / Dt->tp, t2 = task % Dt->tp;
    int ps = orc_pp_owner(S, m->L, l), pd = orc_pp_owner(Dt, m->L, l);
    const uint8_t* sslab[64];
    int64_t snb[64];
    uint8_t* dslab[64];
    int64_t dnb[64];
    for (int t = 0; t < S->tp; ++t) {
        int r = orc_rank(S, ps, t);
        snb[t] = J->src_nb[r];
        sslab[t] = J->src[r] + (l - orc_stage_first(S, m->L, ps)) * orc_layer_slab_bytes(S, m, snb[t]);
    }
    for (int t = 0; t < Dt->tp; ++t) {
        int r = orc_rank(Dt, pd, t);
        dnb[t] = J->dst_nb[r];
        dslab[t] = J->dst[r] + (l - orc_stage_first(Dt, m->L, pd)) * orc_layer_slab_bytes(Dt, m, dnb[t]);
    }
    return orc_migrate_layer_ex(S, Dt, m, J->n_seq, J->maxb, J->lens, J->bt, J->dst_bt, sslab, snb, dslab, dnb, t2,
                                t2 + 1, J->mode, J->src_layout, J->dst_layout, J->valid_only);
}

static void* worker(void* arg) {
    job_t* J = (job_t*)arg;
    int ntask = (J->layer_hi - J->layer_lo) * J->Dt->tp;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int task = J->next_task++;
        pthread_mutex_unlock(&J->mu);
        if (task >= ntask) break;
        int rc = run_task(J, task);
        if (rc) {
            pthread_mutex_lock(&J->mu);
            J->rc = rc;
            pthread_mutex_unlock(&J->mu);
        }
    }
    return NULL;
}

int orc_migrate_ex(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb,
                   const int32_t* lens, const int32_t* bt, const int32_t* dst_bt, const uint8_t* const* src,
                   const int64_t* src_nb, uint8_t* const* dst, const int64_t* dst_nb, int mode, int nthreads,
                   int layer_lo, int layer_hi, int src_layout, int dst_layout, int valid_only) {
    if (orc_topo_check(S, m) || orc_topo_check(Dt, m) || S->tp > 64 || Dt->tp > 64) return -2;
    job_t J = {S, Dt, m, n_seq, maxb, lens, bt, dst_bt, src, src_nb, dst, dst_nb, mode, layer_lo, layer_hi,
               src_layout, dst_layout, valid_only, 0, 0, PTHREAD_MUTEX_INITIALIZER};
    if (nthreads <= 1) {
        worker(&J);
    } else {
        pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)nthreads);
        for (int i = 0; i < nthreads; ++i) pthread_create(&th[i], NULL, worker, &J);
        for (int i = 0; i < nthreads; ++i) pthread_join(th[i], NULL);
        free(th);
    }
    return J.rc;
}

int orc_migrate_layout(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb,
                       const int32_t* lens, const int32_t* bt, const int32_t* dst_bt, const uint8_t* const* src,
                       const int64_t* src_nb, uint8_t* const* dst, const int64_t* dst_nb, int mode, int nthreads,
                       int layer_lo, int layer_hi, int src_layout, int dst_layout) {
    return orc_migrate_ex(S, Dt, m, n_seq, maxb, lens, bt, dst_bt, src, src_nb, dst, dst_nb, mode, nthreads, layer_lo,
                          layer_hi, src_layout, dst_layout, 0);
}

int orc_migrate(const orc_topo* S, const orc_topo* Dt, const orc_shape* m, int n_seq, int maxb, const int32_t* lens,
                const int32_t* bt, const int32_t* dst_bt, const uint8_t* const* src, const int64_t* src_nb,
                uint8_t* const* dst, const int64_t* dst_nb, int mode, int nthreads, int layer_lo, int layer_hi) {
    return orc_migrate_layout(S, Dt, m, n_seq, maxb, lens, bt, dst_bt, src, src_nb, dst, dst_nb, mode, nthreads,
                              layer_lo, layer_hi, 0, 0);
}
