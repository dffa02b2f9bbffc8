"""CPU-only pins of the oracle: what the paper and the mathematics fix, stated without the oracle's code.

Sections cited are the paper's: 3.4.1 (logical model, ownership, preservation law), Algorithm 1 (plan),
3.4.5 (invariants: layer coverage, head coverage, block identity / deterministic remapping, capacity).
"""
import math
import os

import numpy as np
import pytest

from oracle import brute
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import POISON_BYTE, Shape, Topo, make_workload, small_workload
from tests import helpers as H

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _models():
    rows = [l.split() for l in open(os.path.join(GOLD, "model_shapes.txt")) if l.strip() and l[0] != "#"]
    return [(n, int(a), int(b)) for n, a, b in rows]


def _layouts():
    rows = [l.split() for l in open(os.path.join(GOLD, "layouts.txt")) if l.strip() and l[0] != "#"]
    return [Topo(int(a), int(b)) for a, b in rows]


# ---------------------------------------------------------------- ownership (section 3.4.1)

def test_pp_owner_is_a_contiguous_balanced_partition():
    for L in range(1, 13):
        for PP in range(1, L + 1):
            T = Topo(1, PP)
            owners = [orc.pp_owner(T, L, l) for l in range(L)]
            assert owners == sorted(owners) and set(owners) == set(range(PP))      # ascending, all stages used
            sizes = np.bincount(owners, minlength=PP)
            assert sizes.sum() == L and sizes.max() - sizes.min() <= 1
            assert list(sizes) == sorted(sizes, reverse=True)                      # longer stages first
            for p in range(PP + 1):
                assert orc.stage_first(T, L, p) == int(sizes[:p].sum())


def test_pp_owner_explicit_boundaries():
    T = Topo(1, 3, (0, 1, 5, 7))
    assert [orc.pp_owner(T, 7, l) for l in range(7)] == [0, 1, 1, 1, 1, 2, 2]
    m = Shape(7, 2, 8, 4, 2)
    assert orc.topo_check(T, m) == 0
    assert orc.topo_check(Topo(1, 3, (0, 1, 1, 7)), m) != 0       # empty stage
    assert orc.topo_check(Topo(1, 3, (0, 1, 5, 6)), m) != 0       # does not end at L
    assert orc.topo_check(Topo(1, 8), m) != 0                     # more stages than layers


def test_head_coverage_and_replication_multiplicity():
    """Head-coverage invariant: union of TP ranges = [0,H); every head owned exactly rep times."""
    for Hh in (1, 2, 4, 8, 12, 32):
        for TP in range(1, 65):
            T = Topo(TP, 1)
            m = Shape(1, Hh, 8, 4, 2)
            legal = (Hh % TP == 0) if TP <= Hh else (TP % Hh == 0)
            assert (orc.topo_check(T, m) == 0) == legal
            if not legal:
                continue
            rep = max(1, TP // Hh)
            assert orc.rep(T, Hh) == rep and orc.heads_per_rank(T, Hh) == max(1, Hh // TP)
            mult = np.zeros(Hh, dtype=int)
            prev_lo = -1
            for t in range(TP):
                lo, hi = orc.head_range(T, Hh, t)
                assert 0 <= lo < hi <= Hh and hi - lo == max(1, Hh // TP) and lo >= prev_lo
                prev_lo = lo
                mult[lo:hi] += 1
                for h in range(Hh):
                    assert orc.owns_head(T, Hh, t, h) == (lo <= h < hi)
            assert (mult == rep).all()
            for h in range(Hh):
                assert orc.tp_owner(T, Hh, h) == h * rep if TP > Hh else orc.tp_owner(T, Hh, h) == h // (Hh // TP)


def test_rank_linearisation_tp_innermost():
    T = Topo(4, 2)
    assert [orc.rank_of(T, p, t) for p in range(2) for t in range(4)] == list(range(8))


# ---------------------------------------------------------------- Algorithm 1

def _closed_form_items(L, Hh, a, c):
    a1, c1 = min(a, Hh), min(c, Hh)
    return L * (c if c > Hh else a1 + c1 - math.gcd(a1, c1))


@pytest.mark.parametrize("name,L,Hh", _models())
def test_plan_size_closed_form_on_paper_models_and_layouts(name, L, Hh):
    """Overlaps of two even partitions of [0,H) number a+c-gcd(a,c); one item per destination rank when
    heads are replicated on the destination side."""
    m = Shape(L, Hh, 128, 16, 2)
    for S in _layouts():
        for D in _layouts():
            items = orc.plan(S, D, m)
            assert len(items) == _closed_form_items(L, Hh, S.tp, D.tp), (name, S, D)
            # as printed (no de-duplication) a replicated source adds one item per extra replica
            printed = orc.plan(S, D, m, dedupe=False)
            assert len(printed) == len(items) * max(1, S.tp // Hh)


def test_plan_items_cover_each_destination_rank_exactly():
    """Receive side: per layer the items of a destination rank tile its head range with no overlap, come
    from the stage that owns the layer, and from the lowest replica. Send side is the same list grouped
    by source (duality): each source canonical rank sends each of its heads to every owner."""
    for (L, Hh) in ((6, 4), (8, 8), (5, 2)):
        m = Shape(L, Hh, 8, 4, 2)
        topos = [Topo(tp, pp) for tp in (1, 2, 4, 8, 16) for pp in (1, 2, 3, 5) if orc.topo_check(Topo(tp, pp), m) == 0]
        for S in topos:
            for D in topos:
                items = orc.plan(S, D, m)
                recv = {}
                for src, dst, l, lo, hi in items:
                    assert src // S.tp == orc.pp_owner(S, L, l) and dst // D.tp == orc.pp_owner(D, L, l)
                    assert orc.head_range(S, Hh, src % S.tp)[0] <= lo and hi <= orc.head_range(S, Hh, src % S.tp)[1]
                    assert (src % S.tp) % orc.rep(S, Hh) == 0
                    recv.setdefault((dst, l), []).append((lo, hi))
                for p in range(D.pp):
                    for t in range(D.tp):
                        for l in range(orc.stage_first(D, L, p), orc.stage_first(D, L, p + 1)):
                            got = sorted(recv[(p * D.tp + t, l)])
                            want = orc.head_range(D, Hh, t)
                            assert got[0][0] == want[0] and got[-1][1] == want[1]
                            assert all(got[i][1] == got[i + 1][0] for i in range(len(got) - 1))
                sent = np.zeros((L, Hh), dtype=int)
                for src, dst, l, lo, hi in items:
                    sent[l, lo:hi] += 1
                assert (sent == orc.rep(D, Hh)).all()


# ---------------------------------------------------------------- allocation (section 3.4.5, block identity)

def test_alloc_is_exclusive_cumsum_and_compact():
    rng = np.random.default_rng(1)
    for bs in (1, 16, 32):
        lens = rng.integers(0, 200, size=50).astype(np.int32)
        maxb = int(-(-lens.max() // bs)) + 2
        dbt, off, total = orc.alloc(lens, maxb, bs, 7, [10**6, 10**6])
        need = np.ceil(lens / bs).astype(np.int64)
        assert total == need.sum()
        assert (off == np.concatenate([[0], np.cumsum(need)])).all()
        ids = dbt[dbt >= 0]
        assert sorted(ids) == list(range(7, 7 + total))                     # exactly [base, base+total)
        for s in range(len(lens)):
            assert (dbt[s, :need[s]] == 7 + off[s] + np.arange(need[s])).all() and (dbt[s, need[s]:] == -1).all()
        # idempotence: an already compact table allocates to itself
        dbt2, _, _ = orc.alloc(lens, maxb, bs, 7, [10**6])
        assert (dbt2 == dbt).all()


def test_alloc_capacity_and_width_errors():
    lens = np.array([16, 17, 0, 1], dtype=np.int32)          # 1 + 2 + 0 + 1 = 4 blocks
    orc.alloc(lens, 2, 16, 0, [4, 9])
    with pytest.raises(orc.CapacityError):
        orc.alloc(lens, 2, 16, 0, [9, 3])
    with pytest.raises(orc.CapacityError):
        orc.alloc(lens, 2, 16, 1, [4])
    with pytest.raises(ValueError):
        orc.alloc(lens, 1, 16, 0, [99])


# ---------------------------------------------------------------- migration vs numpy slicing

def _run_case(S, D, m, lens, bt, pool, seed, base=0, extra_dst=3, mode="row", nthreads=1):
    G = H.random_global(m, pool, seed)
    src = H.shards_from_global(S, m, G)
    ndst = D.tp * D.pp
    total_need = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [base + total_need + extra_dst + (r % 2) for r in range(ndst)]      # unequal pools on purpose
    dbt, off, total = orc.alloc(lens, bt.shape[1], m.block_size, base, dst_nb)
    dst = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(ndst)])
    rc = orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * (S.tp * S.pp), dst, dst_nb, mode=mode, nthreads=nthreads)
    assert rc == 0
    want = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), base, dst_nb)
    return G, src, dst, want, dbt, dst_nb


TOPOS_H4 = [Topo(1, 1), Topo(2, 1), Topo(1, 2), Topo(2, 2), Topo(4, 1), Topo(8, 1), Topo(4, 3), Topo(16, 2)]


@pytest.mark.parametrize("mode", ["elem", "row"])
def test_all_topology_pairs_equal_numpy_slicing(mode):
    """Every pair of {TP1PP1 ... TP16PP2} on a 6-layer, 4-head model: heads split/merge, replication
    (TP 8 and 16 > 4 heads), layer regrouping with uneven stages (6 layers over 4... 3 stages)."""
    m = Shape(6, 4, 8, 4, 2)
    lens, bt, pool = small_workload(m, 5, 19, seed=3, zero_fraction=0.2)
    for S in TOPOS_H4:
        for D in TOPOS_H4:
            _G, _src, dst, want, _dbt, _nb = _run_case(S, D, m, lens, bt, pool, seed=11, base=2, mode=mode)
            for r in range(len(dst)):
                assert np.array_equal(dst[r], want[r]), (str(S), str(D), r)


def test_identity_topology_identity_table_is_memcpy():
    m = Shape(3, 2, 16, 8, 1)
    lens = np.array([8, 24, 3], dtype=np.int32)
    need = -(-lens // 8)
    bt = np.full((3, 3), -1, dtype=np.int32)
    k = 0
    for s in range(3):
        bt[s, :need[s]] = np.arange(k, k + need[s]); k += need[s]
    T = Topo(2, 1)
    G = H.random_global(m, k, 5)
    src = H.shards_from_global(T, m, G)
    dbt, _, total = orc.alloc(lens, 3, 8, 0, [k, k])
    assert total == k and (dbt == bt).all()
    dst = H.poison_like([b.size for b in src])
    assert orc.migrate(T, T, m, lens, bt, dbt, src, [k, k], dst, [k, k]) == 0
    for a, b in zip(src, dst):
        assert a.tobytes() == b.tobytes()


def test_explicit_uneven_stages():
    m = Shape(7, 2, 8, 4, 2)
    lens, bt, pool = small_workload(m, 4, 15, seed=8)
    S, D = Topo(2, 3, (0, 1, 5, 7)), Topo(1, 2, (0, 6, 7))
    _G, _src, dst, want, _dbt, _nb = _run_case(S, D, m, lens, bt, pool, seed=2)
    for a, b in zip(dst, want):
        assert np.array_equal(a, b)


def test_elem_bytes_1_2_4_and_threads():
    for e in (1, 2, 4):
        m = Shape(4, 4, 8, 4, e)
        lens, bt, pool = small_workload(m, 6, 30, seed=e)
        _G, _src, dst1, want, _dbt, _nb = _run_case(Topo(2, 2), Topo(4, 1), m, lens, bt, pool, seed=e, nthreads=1)
        _G, _src, dst4, _want, _dbt, _nb = _run_case(Topo(2, 2), Topo(4, 1), m, lens, bt, pool, seed=e, nthreads=4)
        for a, b, c in zip(dst1, dst4, want):
            assert np.array_equal(a, c) and np.array_equal(b, c)


def test_layer_window_only_touches_those_layers():
    m = Shape(6, 2, 8, 4, 2)
    lens, bt, pool = small_workload(m, 4, 15, seed=4)
    S, D = Topo(1, 2), Topo(2, 3)
    G = H.random_global(m, pool, 1)
    src = H.shards_from_global(S, m, G)
    nb = [pool + 1] * 6
    dbt, _, total = orc.alloc(lens, bt.shape[1], m.block_size, 0, nb)
    dst = H.poison_like([orc.shard_bytes(D, m, r, nb[r]) for r in range(6)])
    assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * 2, dst, nb, layer_lo=2, layer_hi=4) == 0
    want = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), 0, nb)
    for r in range(6):
        p = r // 2
        if p == 1:      # stage 1 of 3 holds layers 2,3
            assert np.array_equal(dst[r], want[r])
        else:
            assert (dst[r] == POISON_BYTE).all()


def test_replicated_source_reads_lowest_replica():
    """Replicas filled with different bytes: the result must follow the lowest-ranked owner of a head."""
    m = Shape(2, 2, 8, 4, 2)
    lens, bt, pool = small_workload(m, 3, 11, seed=6)
    S, D = Topo(4, 1), Topo(1, 2)         # 4 ranks over 2 heads: ranks {0,1} hold head 0, {2,3} head 1
    G = H.random_global(m, pool, 9)
    src = H.shards_from_global(S, m, G)
    src[1] = (src[1] ^ 0xFF)              # corrupt the non-canonical replicas
    src[3] = (src[3] ^ 0x0F)
    nb = [pool, pool]
    dbt, _, _ = orc.alloc(lens, bt.shape[1], m.block_size, 0, nb)
    dst = H.poison_like([orc.shard_bytes(D, m, r, nb[r]) for r in range(2)])
    assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * 4, dst, nb) == 0
    want = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), 0, nb)
    for a, b in zip(dst, want):
        assert np.array_equal(a, b)


def test_shared_source_block_is_copied_once_per_reference():
    m = Shape(1, 1, 8, 4, 2)
    lens = np.array([8, 8], dtype=np.int32)
    bt = np.array([[5, 2], [5, 0]], dtype=np.int32)            # both sequences start with block 5
    T = Topo(1, 1)
    G = H.random_global(m, 6, 3)
    src = H.shards_from_global(T, m, G)
    dbt, _, _ = orc.alloc(lens, 2, 4, 0, [4])
    dst = H.poison_like([orc.shard_bytes(T, m, 0, 4)])
    assert orc.migrate(T, T, m, lens, bt, dbt, src, [6], dst, [4]) == 0
    want = H.expected_by_slicing(T, m, G, np.array([5, 2, 5, 0]), 0, [4])
    assert np.array_equal(dst[0], want[0])


def test_bad_block_ids_are_reported_and_skipped():
    m = Shape(1, 1, 8, 4, 2)
    lens = np.array([8], dtype=np.int32)
    bt = np.array([[1, 9]], dtype=np.int32)                     # 9 is outside the 3-block source pool
    T = Topo(1, 1)
    G = H.random_global(m, 3, 3)
    src = H.shards_from_global(T, m, G)
    dbt, _, _ = orc.alloc(lens, 2, 4, 0, [2])
    dst = H.poison_like([orc.shard_bytes(T, m, 0, 2)])
    assert orc.migrate(T, T, m, lens, bt, dbt, src, [3], dst, [2]) == -6
    v = brute.shard_view(T, m, 0, dst[0], 2)
    assert np.array_equal(v[:, :, 0], G[:, :, 1]) and (v[:, :, 1] == POISON_BYTE).all()


# ---------------------------------------------------------------- brute force, exactly-once, byte counts

def test_tiny_workload_brute_force_exactly_once_and_round_trip():
    """The Tiny benchmark configuration, TP1PP1 -> TP2PP2 -> TP1PP1, enumerated element by element."""
    w = make_workload("tiny")
    m = w.shape
    assert (w.seq_lens >= 1).all() and (w.seq_lens <= 256).all() and w.num_seqs == 8
    assert sorted(w.block_tables[w.block_tables >= 0]) == list(range(w.num_src_blocks))    # a permutation
    A, B = w.chain[0], w.chain[1]
    G = H.random_global(m, w.num_src_blocks, 0)
    src = H.shards_from_global(A, m, G)
    nbB = [w.live_blocks] * 4
    dbt, _, total = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, nbB)
    before = H.poison_like([orc.shard_bytes(B, m, r, nbB[r]) for r in range(4)])
    mid = [b.copy() for b in before]
    assert orc.migrate(A, B, m, w.seq_lens, w.block_tables, dbt, src, [w.num_src_blocks], mid, nbB, mode="elem") == 0
    res = brute.enumerate_check(A, B, m, w.seq_lens, w.block_tables, dbt, src, [w.num_src_blocks], mid, nbB, before)
    assert res == {"mismatched_bytes": 0, "unowned_rows": 0, "not_exactly_once": 0, "stray_writes": 0}
    # byte count closed form: W = NB_live * L * 2 * H * rep * bs * D * e
    assert sum(b.size for b in mid) == total * m.num_layers * 2 * m.num_kv_heads * m.block_size * m.head_dim * m.elem_bytes
    # and back
    nbA = [total]
    dbt2, _, _ = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, nbA)
    back_before = H.poison_like([orc.shard_bytes(A, m, 0, total)])
    back = [b.copy() for b in back_before]
    assert orc.migrate(B, A, m, w.seq_lens, dbt, dbt2, mid, nbB, back, nbA, mode="elem") == 0
    res = brute.enumerate_check(B, A, m, w.seq_lens, dbt, dbt2, mid, nbB, back, nbA, back_before)
    assert not any(res.values())
    # logical content is preserved; physically it equals the identity-topology (defragmenting) migration
    assert np.array_equal(brute.logical_dump(A, m, src, [w.num_src_blocks], w.seq_lens, w.block_tables),
                          brute.logical_dump(A, m, back, nbA, w.seq_lens, dbt2))
    ident = [b.copy() for b in back_before]
    assert orc.migrate(A, A, m, w.seq_lens, w.block_tables, dbt2, src, [w.num_src_blocks], ident, nbA) == 0
    assert np.array_equal(ident[0], back[0])


def test_brute_force_with_replication_counts_once_per_replica():
    m = Shape(3, 2, 8, 4, 2)
    lens, bt, pool = small_workload(m, 4, 14, seed=12, zero_fraction=0.25)
    for S, D in ((Topo(1, 3), Topo(4, 1)), (Topo(4, 1), Topo(2, 3)), (Topo(8, 1), Topo(4, 3))):
        G = H.random_global(m, pool, 4)
        src = H.shards_from_global(S, m, G)
        nd = D.tp * D.pp
        total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
        nb = [total + 2] * nd
        dbt, _, _ = orc.alloc(lens, bt.shape[1], m.block_size, 1, nb)
        before = H.poison_like([orc.shard_bytes(D, m, r, nb[r]) for r in range(nd)])
        after = [b.copy() for b in before]
        assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * (S.tp * S.pp), after, nb, mode="elem") == 0
        res = brute.enumerate_check(S, D, m, lens, bt, dbt, src, [pool] * (S.tp * S.pp), after, nb, before)
        assert not any(res.values()), (str(S), str(D), res)
        assert brute.replicas_consistent(D, m, after, nb)
        written = sum(int((a != b).sum()) for a, b in zip(after, before))
        W = total * m.num_layers * 2 * m.num_kv_heads * orc.rep(D, m.num_kv_heads) * m.block_size * m.head_dim * m.elem_bytes
        assert 0.97 * W <= written <= W          # random bytes equal the poison value 1/256 of the time


def test_round_trips_over_topology_pairs_preserve_logical_content():
    m = Shape(4, 4, 8, 4, 2)
    lens, bt, pool = small_workload(m, 5, 21, seed=21)
    topos = [Topo(1, 1), Topo(2, 1), Topo(1, 2), Topo(2, 2), Topo(4, 1), Topo(8, 1)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    for A in topos:
        G = H.random_global(m, pool, 2)
        srcA = H.shards_from_global(A, m, G)
        dumpA = brute.logical_dump(A, m, srcA, [pool] * (A.tp * A.pp), lens, bt)
        for B in topos:
            nbB = [total] * (B.tp * B.pp)
            dbtB, _, _ = orc.alloc(lens, bt.shape[1], m.block_size, 0, nbB)
            midB = H.poison_like([orc.shard_bytes(B, m, r, total) for r in range(B.tp * B.pp)])
            assert orc.migrate(A, B, m, lens, bt, dbtB, srcA, [pool] * (A.tp * A.pp), midB, nbB) == 0
            assert np.array_equal(brute.logical_dump(B, m, midB, nbB, lens, dbtB), dumpA)
            nbA = [total] * (A.tp * A.pp)
            dbtA, _, _ = orc.alloc(lens, bt.shape[1], m.block_size, 0, nbA)
            back = H.poison_like([orc.shard_bytes(A, m, r, total) for r in range(A.tp * A.pp)])
            assert orc.migrate(B, A, m, lens, dbtB, dbtA, midB, nbB, back, nbA) == 0
            ident = H.poison_like([orc.shard_bytes(A, m, r, total) for r in range(A.tp * A.pp)])
            assert orc.migrate(A, A, m, lens, bt, dbtA, srcA, [pool] * (A.tp * A.pp), ident, nbA) == 0
            for x, y in zip(back, ident):
                assert np.array_equal(x, y)


def test_offsets_match_numpy_strides():
    """The oracle's byte offsets are those of a dense row-major [l][2][nb][hl][bs][D] array."""
    m = Shape(5, 4, 8, 4, 2)
    T = Topo(2, 2)
    nb = 3
    for rank in range(4):
        p, t = divmod(rank, 2)
        nl = 3 if p == 0 else 2
        arr = np.zeros((nl, 2, nb, 2, 4, 8), dtype=np.uint16)
        assert orc.shard_bytes(T, m, rank, nb) == arr.nbytes
        for (l, kv, b, h, tok, d) in ((0, 0, 0, 0, 0, 0), (1, 1, 2, 1, 3, 7), (nl - 1, 0, 1, 0, 2, 5)):
            gl, gh = l + (0 if p == 0 else 3), h + 2 * t
            want = sum(i * s for i, s in zip((l, kv, b, h, tok, d), arr.strides))
            assert orc.offset(T, m, rank, nb, gl, kv, b, gh, tok, d) == want
        assert orc.offset(T, m, rank, nb, 0 if p == 1 else 4, 0, 0, 2 * t) == -1     # layer of the other stage
        assert orc.offset(T, m, rank, nb, 3 * p, 0, 0, 2 * (1 - t)) == -1             # head of the other rank


# ---------------------------------------------------------------- capacity constraint (section 3.4.5)

def test_preemption_keeps_longest_fitting_prefix():
    """Kept set = {s : cumsum(need)[s] <= avail} (numpy), a prefix; maximal (the first preempted sequence
    does not fit); ids of kept sequences are those of the unconstrained allocator; with enough room nothing
    is preempted; brute force over every prefix on tiny cases."""
    rng = np.random.default_rng(9)
    for trial in range(60):
        n = int(rng.integers(1, 12))
        bs = int(rng.choice([1, 4, 16]))
        lens = rng.integers(0, 70, size=n).astype(np.int32)
        need = -(-lens.astype(np.int64) // bs)
        maxb = int(need.max()) + 1
        base = int(rng.integers(0, 4))
        caps = [base + int(rng.integers(0, need.sum() + 3)), base + int(need.sum()) + 5]
        avail = min(caps) - base
        dbt, pre, total = orc.alloc_preempt(lens, maxb, bs, base, caps)
        kept = np.cumsum(need) <= avail
        assert np.array_equal(pre, (~kept).astype(np.int32))
        assert not kept[np.argmin(kept):].any() if not kept.all() else True          # a prefix
        assert total == int(need[kept].sum()) <= avail
        if not kept.all():
            first = int(np.argmin(kept))
            assert total + need[first] > avail                                        # maximal
        # brute force: the longest prefix whose blocks fit
        best = max(k for k in range(n + 1) if need[:k].sum() <= avail)
        assert int(kept.sum()) == best
        ref_bt, _off, _tot = orc.alloc(np.where(kept, lens, 0).astype(np.int32), maxb, bs, base, [10**9])
        assert np.array_equal(dbt, ref_bt)
        if kept.all():
            full_bt, _o, full_total = orc.alloc(lens, maxb, bs, base, caps)
            assert np.array_equal(dbt, full_bt) and total == full_total


# ---------------------------------------------------------------- token-major block layout

def _to_token_major(T, m, shards, nb):
    """numpy transpose of every rank's [l][2][nb][hl][bs][De] array to [l][2][nb][bs][hl][De]."""
    out = []
    for r, b in enumerate(shards):
        v = brute.shard_view(T, m, r, b, nb[r] if isinstance(nb, (list, tuple)) else nb)
        out.append(np.ascontiguousarray(v.transpose(0, 1, 2, 4, 3, 5)).reshape(-1))
    return out


@pytest.mark.parametrize("src_layout,dst_layout", [("token", "token"), ("token", "head"), ("head", "token")])
def test_token_major_layouts_are_transposes_of_the_canonical_result(src_layout, dst_layout):
    """[block][token][head][dim] on either side: the result is the numpy transpose of the head-major one."""
    m = Shape(4, 4, 8, 4, 2)
    lens, bt, pool = small_workload(m, 5, 19, seed=31, zero_fraction=0.2)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    for S in (Topo(1, 1), Topo(2, 2), Topo(4, 1), Topo(8, 1)):
        for D in (Topo(1, 2), Topo(2, 1), Topo(4, 4), Topo(8, 1)):
            G = H.random_global(m, pool, 5)
            src = H.shards_from_global(S, m, G)
            nd = D.tp * D.pp
            nb = [total + 1 + (r % 2) for r in range(nd)]
            want = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), 0, nb)
            if src_layout == "token":
                src = _to_token_major(S, m, src, pool)
            if dst_layout == "token":
                want = _to_token_major(D, m, want, nb)
            dbt, _off, _t = orc.alloc(lens, bt.shape[1], m.block_size, 0, nb)
            for mode in ("elem", "row"):
                dst = H.poison_like([w_.size for w_ in want])
                assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * len(src), dst, nb, mode=mode,
                                   src_layout=src_layout, dst_layout=dst_layout) == 0
                for a, b in zip(dst, want):
                    assert np.array_equal(a, b), (str(S), str(D), mode)


# ---------------------------------------------------------------- shared prefixes (section 3.4.5)

def _shared_tables(rng, n, bs, pool, max_len, share):
    """Random tables in which sequences reuse the leading blocks of earlier sequences (shared prefixes)."""
    lens = rng.integers(0, max_len + 1, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // bs)
    maxb = int(need.max(initial=1)) + 1
    bt = np.full((n, maxb), -1, dtype=np.int32)
    free = list(rng.permutation(pool))
    for s in range(n):
        k = 0
        if s and rng.random() < share:                      # share a prefix with an earlier sequence
            o = int(rng.integers(0, s))
            k = int(rng.integers(0, min(need[s], need[o]) + 1))
            bt[s, :k] = bt[o, :k]
        for j in range(k, need[s]):
            bt[s, j] = free.pop()
    return lens, bt


def test_shared_allocation_preserves_sharing_and_matches_numpy_unique():
    rng = np.random.default_rng(77)
    for trial in range(40):
        bs = int(rng.choice([4, 16]))
        pool = 400
        lens, bt = _shared_tables(rng, int(rng.integers(1, 14)), bs, pool, 100, share=0.6)
        flat = H.flat_live_ids(Shape(1, 1, 8, bs, 2), lens, bt)
        base = int(rng.integers(0, 5))
        dbt, total, bad = orc.alloc_shared(lens, bt, bs, base, pool, [10**6])
        assert not bad
        # numpy statement: ids by order of first occurrence of each distinct source id
        uniq, first_idx, inverse = np.unique(flat, return_index=True, return_inverse=True)
        order = np.argsort(np.argsort(first_idx))            # rank of each distinct id by first occurrence
        want_flat = base + order[inverse]
        need = -(-lens.astype(np.int64) // bs)
        got_flat = np.concatenate([dbt[s, :need[s]] for s in range(len(lens))] + [np.zeros(0, np.int32)])
        assert total == len(uniq) and np.array_equal(got_flat, want_flat)
        for s in range(len(lens)):
            assert (dbt[s, need[s]:] == -1).all()
        # equal source <=> equal destination; ids are exactly [base, base+total)
        assert sorted(set(got_flat.tolist())) == list(range(base, base + total))
        for a in range(len(flat)):
            for b in range(a + 1, len(flat)):
                assert (flat[a] == flat[b]) == (got_flat[a] == got_flat[b])
        # without sharing it is the plain allocator
        if len(uniq) == len(flat):
            plain, _off, ptotal = orc.alloc(lens, bt.shape[1], bs, base, [10**6])
            assert np.array_equal(plain, dbt) and ptotal == total
    # capacity counts distinct blocks; out-of-pool ids get their own block and are reported
    lens = np.array([8, 8], dtype=np.int32)
    bt = np.array([[3, 5], [3, 9]], dtype=np.int32)
    dbt, total, bad = orc.alloc_shared(lens, bt, 4, 0, 10, [3])
    assert total == 3 and not bad and dbt.tolist() == [[0, 1], [0, 2]]
    with pytest.raises(orc.CapacityError):
        orc.alloc_shared(lens, bt, 4, 0, 10, [2])
    dbt, total, bad = orc.alloc_shared(lens, np.array([[3, 50], [3, -4]], dtype=np.int32), 4, 0, 10, [9])
    assert bad and total == 3 and dbt.tolist() == [[0, 1], [0, 2]]


def test_shared_allocation_migrates_each_distinct_block_once():
    """Content seen through the rewritten tables equals the content seen through the old ones."""
    m = Shape(2, 2, 8, 4, 2)
    rng = np.random.default_rng(5)
    pool = 60
    lens, bt = _shared_tables(rng, 6, m.block_size, pool, 40, share=0.8)
    S, D = Topo(1, 2), Topo(2, 1)
    G = H.random_global(m, pool, 8)
    src = H.shards_from_global(S, m, G)
    dbt, total, _bad = orc.alloc_shared(lens, bt, m.block_size, 0, pool, [total_ := 10**6] * 2)
    flat = H.flat_live_ids(m, lens, bt)
    assert total == len(set(flat.tolist())) < len(flat)
    nb = [total, total]
    dst = H.poison_like([orc.shard_bytes(D, m, r, total) for r in range(2)])
    assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * 2, dst, nb) == 0
    assert np.array_equal(brute.logical_dump(S, m, src, [pool] * 2, lens, bt),
                          brute.logical_dump(D, m, dst, nb, lens, dbt))
    assert not any((d == POISON_BYTE).all() for d in dst)


# ---------------------------------------------------------------- valid tokens only

@pytest.mark.parametrize("layout", ["head", "token"])
def test_valid_tokens_only_masks_the_slack_of_partial_blocks(layout):
    """With valid_only the result equals the whole-block result where a token slot is in use and the poison
    fill elsewhere (numpy mask over the token axis of every sequence's last block)."""
    m = Shape(3, 4, 8, 4, 2)
    lens, bt, pool = small_workload(m, 7, 23, seed=51, zero_fraction=0.15)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    for S, D in ((Topo(1, 1), Topo(2, 3)), (Topo(4, 1), Topo(2, 1)), (Topo(2, 1), Topo(8, 1))):
        G = H.random_global(m, pool, 6)
        src = H.shards_from_global(S, m, G)
        nd = D.tp * D.pp
        nb = [total + 2] * nd
        full = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), 1, nb)
        dbt, off, _t = orc.alloc(lens, bt.shape[1], m.block_size, 1, nb)
        # slack mask per destination block id: tokens >= valid count keep the poison
        used = np.zeros((nb[0], m.block_size), dtype=bool)
        for s, n in enumerate(lens):
            for j in range(-(-int(n) // m.block_size)):
                used[dbt[s, j], :min(m.block_size, int(n) - j * m.block_size)] = True
        want = []
        for r in range(nd):
            v = brute.shard_view(D, m, r, full[r].copy(), nb[r])          # [l][2][nb][hl][bs][De]
            v[:, :, ~used.any(axis=1)] = POISON_BYTE
            mask = ~used[None, None, :, None, :, None]
            v[np.broadcast_to(mask, v.shape)] = POISON_BYTE
            want.append(v.reshape(-1))
        if layout == "token":
            src = _to_token_major(S, m, src, pool)
            want = _to_token_major(D, m, want, nb)
        for mode in ("elem", "row"):
            dst = H.poison_like([w_.size for w_ in want])
            assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * len(src), dst, nb, mode=mode, src_layout=layout,
                               dst_layout=layout, valid_only=True) == 0
            for a, b in zip(dst, want):
                assert np.array_equal(a, b), (str(S), str(D), mode)


def test_round_trip_from_a_compact_table_reproduces_the_input_bytes():
    """A -> B -> A with A's table already compact and in order: every pool byte comes back (bit for bit)."""
    m = Shape(4, 4, 8, 4, 2)
    lens = np.array([9, 0, 4, 17, 1], dtype=np.int32)
    need = -(-lens.astype(np.int64) // m.block_size)
    total = int(need.sum())
    bt, _off, _t = orc.alloc(lens, int(need.max()) + 1, m.block_size, 0, [total])     # compact, in order
    for A in (Topo(1, 1), Topo(2, 2), Topo(4, 1), Topo(8, 2)):
        G = H.random_global(m, total, 13)
        src = H.shards_from_global(A, m, G)
        na = A.tp * A.pp
        for B in (Topo(1, 4), Topo(2, 1), Topo(4, 2), Topo(16, 1)):
            nb = B.tp * B.pp
            dbt, _o, _t2 = orc.alloc(lens, bt.shape[1], m.block_size, 0, [total] * nb)
            assert np.array_equal(dbt, bt)
            mid = H.poison_like([orc.shard_bytes(B, m, r, total) for r in range(nb)])
            assert orc.migrate(A, B, m, lens, bt, dbt, src, [total] * na, mid, [total] * nb) == 0
            back = H.poison_like([b.size for b in src])
            assert orc.migrate(B, A, m, lens, dbt, bt, mid, [total] * nb, back, [total] * na) == 0
            for a, b in zip(src, back):
                assert a.tobytes() == b.tobytes(), (str(A), str(B))


def test_brute_force_enumerator_catches_each_kind_of_damage():
    """Negative controls for the checker itself: a flipped byte, a block that was never copied, two live
    blocks sent to one destination block and a write into a slack block each raise their own counter."""
    m = Shape(2, 2, 8, 4, 2)
    A, B = Topo(1, 1), Topo(2, 2)
    lens, bt, pool = small_workload(m, 4, 14, seed=21, zero_fraction=0.0)
    G = H.random_global(m, pool, 4)
    src = H.shards_from_global(A, m, G)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    nb = [total + 2] * 4                                  # two slack blocks per destination pool
    dbt, _, _ = orc.alloc(lens, bt.shape[1], m.block_size, 0, nb)
    before = H.poison_like([orc.shard_bytes(B, m, r, nb[r]) for r in range(4)])
    good = [b.copy() for b in before]
    assert orc.migrate(A, B, m, lens, bt, dbt, src, [pool], good, nb) == 0
    clean = {"mismatched_bytes": 0, "unowned_rows": 0, "not_exactly_once": 0, "stray_writes": 0}
    assert brute.enumerate_check(A, B, m, lens, bt, dbt, src, [pool], good, nb, before) == clean
    hs = m.block_size * m.head_dim * m.elem_bytes
    # (1) one flipped byte inside a live block
    bad = [b.copy() for b in good]
    bad[3][5] ^= 0x40
    res = brute.enumerate_check(A, B, m, lens, bt, dbt, src, [pool], bad, nb, before)
    assert res["mismatched_bytes"] == 1 and res["not_exactly_once"] == 0 and res["stray_writes"] == 0
    # (2) a live block whose copy never happened (still the fill byte) on one rank, one plane
    bad = [b.copy() for b in good]
    v = brute.shard_view(B, m, 1, bad[1], nb[1])
    v[0, 1, total - 1] = POISON_BYTE
    res = brute.enumerate_check(A, B, m, lens, bt, dbt, src, [pool], bad, nb, before)
    assert res["mismatched_bytes"] > hs // 2 and res["stray_writes"] == 0
    # (3) a table that sends two live blocks to the same destination block
    dup = dbt.copy()
    dup[0, 1] = dup[0, 0]
    res = brute.enumerate_check(A, B, m, lens, bt, dup, src, [pool], good, nb, before)
    assert res["not_exactly_once"] > 0
    # (4) a write into a slack block
    bad = [b.copy() for b in good]
    v = brute.shard_view(B, m, 2, bad[2], nb[2])
    v[0, 0, total + 1, 0, 2, 3] ^= 0xFF
    res = brute.enumerate_check(A, B, m, lens, bt, dbt, src, [pool], bad, nb, before)
    assert res["stray_writes"] == 1 and res["mismatched_bytes"] == 0


# ---------------------------------------------------------------- ranks spread over several devices

def _device_maps(S, D, ndev, kind):
    ns, nd = S.tp * S.pp, D.tp * D.pp
    if kind == "block":                                  # consecutive ranks share a device
        return [r * ndev // ns for r in range(ns)], [r * ndev // nd for r in range(nd)]
    return [r % ndev for r in range(ns)], [(r + 1) % ndev for r in range(nd)]   # interleaved, shifted


@pytest.mark.parametrize("ndev", [1, 2, 4, 8])
@pytest.mark.parametrize("kind", ["block", "interleaved"])
def test_partition_send_and_receive_sides_mirror_each_other(ndev, kind):
    """Section 3.4.2: the send side is the receive side regrouped by source. Over all devices the remote
    receive items and the send items are the same multiset, bytes sent equal bytes received, every item is
    received exactly once, and what a device receives tiles the head ranges of exactly its own ranks."""
    for (L, Hh) in ((80, 8), (32, 32), (48, 4), (6, 4)):
        m = Shape(L, Hh, 128, 16, 2)
        topos = [T for T in _layouts() + [Topo(16, 1), Topo(2, 3)] if orc.topo_check(T, m) == 0]
        for S in topos:
            for D in topos:
                sdev, ddev = _device_maps(S, D, ndev, kind)
                items = orc.plan(S, D, m)
                all_recv, all_send = [], []
                for q in range(ndev):
                    recv, send = orc.plan_partition(S, D, m, sdev, ddev, q)
                    assert all(ddev[d] == q for d in recv[:, 1])
                    assert all(sdev[s] == q and ddev[d] != q for s, d in send[:, :2])
                    assert all(row[5] == sdev[row[0]] for row in recv) and all(row[5] == ddev[row[1]] for row in send)
                    all_recv.append(recv)
                    all_send.append(send)
                    # what q receives covers each (local destination rank, layer of its stage) head range exactly
                    cover = {}
                    for s_, d_, l_, lo, hi, _o in recv:
                        cover.setdefault((int(d_), int(l_)), []).append((int(lo), int(hi)))
                    for d_ in range(D.tp * D.pp):
                        p, t = divmod(d_, D.tp)
                        for l_ in range(orc.stage_first(D, L, p), orc.stage_first(D, L, p + 1)):
                            if ddev[d_] != q:
                                assert (d_, l_) not in cover
                                continue
                            got = sorted(cover[(d_, l_)])
                            want = orc.head_range(D, Hh, t)
                            assert got[0][0] == want[0] and got[-1][1] == want[1]
                            assert all(got[i][1] == got[i + 1][0] for i in range(len(got) - 1))
                recv = np.concatenate(all_recv)
                send = np.concatenate(all_send)
                assert sorted(map(tuple, recv[:, :5])) == sorted(map(tuple, items))          # each item once
                remote = recv[recv[:, 5] != np.asarray(ddev)[recv[:, 1]]]
                assert sorted(map(tuple, remote[:, :5])) == sorted(map(tuple, send[:, :5]))  # duality
                heads = lambda rows: int((rows[:, 4] - rows[:, 3]).sum())
                assert heads(remote) == heads(send)                                          # bytes in == bytes out
                if ndev == 1:
                    assert len(send) == 0
