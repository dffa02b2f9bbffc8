"""GPU parity: the CUDA path through the C ABI against the CPU oracle, bit for bit (pools, tables, ids)."""
import numpy as np
import pytest
import torch

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import POISON_BYTE, Shape, Topo, make_workload, small_workload
from tests import helpers as H
from tests.gpu_harness import gpu_migrate, to_dev

pytestmark = pytest.mark.gpu


def oracle_run(S, D, m, lens, bt, src, src_nb, dst_nb, base=0, mode="row", nthreads=4):
    dbt, off, total = orc.alloc(lens, bt.shape[1], m.block_size, base, dst_nb)
    dst = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(D.tp * D.pp)])
    rc = orc.migrate(S, D, m, lens, bt, dbt, src, src_nb, dst, dst_nb, mode=mode, nthreads=nthreads)
    return dst, dbt, total, rc


def assert_same(got, want_dst, want_dbt, want_total, tag=""):
    assert got["status"] == remp.REMP_OK, tag
    assert got["total"] == want_total, tag
    assert np.array_equal(got["dst_bt"], want_dbt), tag
    for r, (a, b) in enumerate(zip(got["dst"], want_dst)):
        assert a.shape == b.shape and np.array_equal(a, b), (tag, r)


TOPOS_H4 = [Topo(1, 1), Topo(2, 1), Topo(1, 2), Topo(2, 2), Topo(4, 1), Topo(8, 1), Topo(4, 3), Topo(16, 2)]


def test_all_topology_pairs_small():
    m = Shape(6, 4, 8, 4, 2)                       # 64-byte head slices: every chunk is a ragged tail
    lens, bt, pool = small_workload(m, 5, 19, seed=3, zero_fraction=0.2)
    G = H.random_global(m, pool, 11)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    for S in TOPOS_H4:
        src = H.shards_from_global(S, m, G)
        for D in TOPOS_H4:
            nd = D.tp * D.pp
            dst_nb = [2 + total + 3 + (r % 2) for r in range(nd)]
            want = oracle_run(S, D, m, lens, bt, src, [pool] * len(src), dst_nb, base=2)
            got = gpu_migrate(S, D, m, lens, bt, src, [pool] * len(src), dst_nb, base=2)
            assert_same(got, *want[:3], tag=(str(S), str(D)))
            for a, b in zip(got["src_after"], src):
                assert np.array_equal(a, b)          # the source is never written


def test_tiny_config_chain_and_round_trip():
    """Two chains side by side: the oracle's (fed with its own previous result) and the GPU's (fed with its
    own); they must agree after every leg."""
    w = make_workload("tiny")
    m = w.shape
    G = H.random_global(m, w.num_src_blocks, 0)
    o_cur = H.shards_from_global(w.chain[0], m, G)
    g_cur = [b.copy() for b in o_cur]
    cur_nb, o_bt, g_bt = [w.num_src_blocks], w.block_tables, w.block_tables
    for S, D in zip(w.chain[:-1], w.chain[1:]):
        dst_nb = [w.live_blocks] * (D.tp * D.pp)
        want = oracle_run(S, D, m, w.seq_lens, o_bt, o_cur, cur_nb, dst_nb)
        got = gpu_migrate(S, D, m, w.seq_lens, g_bt, g_cur, cur_nb, dst_nb)
        assert_same(got, *want[:3], tag=(str(S), str(D)))
        o_cur, o_bt = want[0], want[1]
        g_cur, g_bt, cur_nb = got["dst"], got["dst_bt"], dst_nb
    # A -> B -> A equals the identity-topology (defragmenting) migration of A
    A = w.chain[0]
    ident = gpu_migrate(A, A, m, w.seq_lens, w.block_tables, H.shards_from_global(A, m, G), [w.num_src_blocks],
                        [w.live_blocks])
    assert np.array_equal(ident["dst"][0], g_cur[0]) and np.array_equal(ident["dst_bt"], g_bt)


@pytest.mark.parametrize("shape,S,D", [
    (Shape(4, 8, 128, 16, 2), Topo(1, 1), Topo(2, 1)),        # 32 KiB runs: 8 full chunks per run
    (Shape(4, 8, 128, 16, 2), Topo(4, 2), Topo(8, 1)),        # 4 KiB runs
    (Shape(4, 8, 128, 16, 2), Topo(8, 1), Topo(2, 4)),        # merge 4 sources per destination block
    (Shape(3, 8, 128, 32, 1), Topo(2, 1), Topo(16, 1)),       # fp8-sized elements, 2x replication
    (Shape(3, 8, 128, 32, 1), Topo(16, 1), Topo(1, 3)),       # replicated source
    (Shape(5, 4, 80, 16, 1), Topo(2, 1), Topo(1, 5)),         # 1280-byte head slices: 2.5 KiB runs, ragged chunk
    (Shape(5, 6, 72, 16, 4), Topo(3, 1), Topo(2, 1)),         # 4608-byte slices, 3 heads vs 2 heads per rank: 1-head runs
    (Shape(7, 2, 64, 8, 2), Topo(2, 3, (0, 1, 5, 7)), Topo(1, 2, (0, 6, 7))),
    (Shape(3, 4, 24, 8, 1), Topo(1, 1), Topo(4, 1)),          # 192-byte head slices: not a power of two (row kernel, block groups)
    (Shape(3, 4, 40, 2, 2), Topo(4, 1), Topo(2, 2)),          # 160-byte slices, 2-head runs of 320 bytes
    (Shape(3, 8, 64, 8, 1), Topo(4, 1), Topo(8, 1)),          # 512-byte slices: groups of 8 blocks per item
    (Shape(3, 8, 128, 1, 2), Topo(4, 1), Topo(8, 1)),         # block_size 1: 256-byte slices, groups of 16 blocks
    (Shape(3, 8, 16, 1, 1), Topo(2, 1), Topo(16, 1)),         # 16-byte slices, 2x replication: groups of 32 blocks
    (Shape(3, 6, 128, 1, 2), Topo(1, 1), Topo(2, 1)),         # 768-byte runs (3 heads): groups of 5 blocks
    (Shape(3, 12, 64, 1, 2), Topo(1, 1), Topo(4, 1)),         # 384-byte runs: groups of 10 blocks
    (Shape(3, 6, 24, 1, 2), Topo(1, 1), Topo(2, 1)),          # 144-byte runs: groups of 28 blocks (block index above 15)
    (Shape(3, 8, 80, 16, 1), Topo(4, 1), Topo(8, 1)),         # 1280-byte runs: groups of 3 blocks
    (Shape(3, 8, 96, 8, 2), Topo(4, 1), Topo(8, 1)),          # 1536-byte runs: one block per item, ragged 2 KiB chunk
])
@pytest.mark.parametrize("opts", [
    {}, {remp.REMP_OPT_CHUNK_BYTES: 1024}, {remp.REMP_OPT_CHUNK_BYTES: 8192},
    {remp.REMP_OPT_CTAS_PER_SM: 8}, {remp.REMP_OPT_TILE_ITEMS: 64}, {remp.REMP_OPT_TILE_ITEMS: 1 << 20},
    {remp.REMP_OPT_SCHEDULE: 1}, {remp.REMP_OPT_SCHEDULE: 1, remp.REMP_OPT_TILE_ITEMS: 100},
    {remp.REMP_OPT_SCHEDULE: 3}, {remp.REMP_OPT_SCHEDULE: 3, remp.REMP_OPT_TILE_ITEMS: 5},
    {remp.REMP_OPT_VEC_BYTES: 32}, {remp.REMP_OPT_VEC_BYTES: 32, remp.REMP_OPT_CHUNK_BYTES: 2048},
    {remp.REMP_OPT_KERNEL: 2}, {remp.REMP_OPT_KERNEL: 2, remp.REMP_OPT_LANES_PER_WARP: 32},
    {remp.REMP_OPT_KERNEL: 2, remp.REMP_OPT_CHUNK_BYTES: 1024, remp.REMP_OPT_CTAS_PER_SM: 2},
    {remp.REMP_OPT_KERNEL: 2, remp.REMP_OPT_CHUNK_BYTES: 16384, remp.REMP_OPT_LANES_PER_WARP: 1},
], ids=lambda o: "-".join(f"{k}={v}" for k, v in o.items()) or "default")
def test_medium_cases_span_many_chunks(shape, S, D, opts):
    m = shape
    lens, bt, pool = small_workload(m, 40, 300, seed=5, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    src = []
    rng = np.random.default_rng(7)
    for r in range(ns):
        src.append(rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8))
    if S.tp > m.num_kv_heads:          # replicas differ on purpose: the lowest owner must win
        pass
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 5] * nd
    want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=3)
    got = gpu_migrate(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=3, options=opts)
    assert_same(got, *want[:3], tag=(str(S), str(D), opts))


def test_strided_shards_match_dense():
    """Non-canonical layer/K-V/block strides (pools embedded in larger allocations)."""
    m = Shape(4, 4, 64, 16, 2)
    S, D = Topo(2, 2), Topo(4, 1)
    lens, bt, pool = small_workload(m, 12, 100, seed=9)
    G = H.random_global(m, pool, 1)
    src = H.shards_from_global(S, m, G)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 1] * 4
    want = oracle_run(S, D, m, lens, bt, src, [pool] * 4, dst_nb)
    hs = m.block_size * m.head_dim * m.elem_bytes
    # source: [layer][block][K,V][head]... layout => stride_block = 2*Hl*hs, stride_kv = Hl*hs
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src, strides = [], []
    for r in range(4):
        v = src[r].reshape(2, 2, pool, 2, hs)                  # [l][kv][blk][hl][hs]
        v = np.ascontiguousarray(v.transpose(0, 2, 1, 3, 4))   # [l][blk][kv][hl][hs]
        d_src.append(to_dev(v.reshape(-1)))
        strides.append({"layer": pool * 2 * 2 * hs, "block": 2 * 2 * hs, "kv": 2 * hs})
    # destination: dense but with padded layer stride
    pad = 4096
    d_dst, dstr = [], []
    for r in range(4):
        layer_bytes = 2 * dst_nb[r] * 1 * hs
        d_dst.append(torch.full((4 * (layer_bytes + pad),), POISON_BYTE, dtype=torch.uint8, device="cuda"))
        dstr.append({"layer": layer_bytes + pad})
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    tot = remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt)
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * 4, strides), remp.make_shards(d_dst, dst_nb, dstr))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    assert tot == want[2]
    for r in range(4):
        layer_bytes = 2 * dst_nb[r] * hs
        g = d_dst[r].cpu().numpy().reshape(4, layer_bytes + pad)
        assert np.array_equal(g[:, :layer_bytes].reshape(-1), want[0][r])
        assert (g[:, layer_bytes:] == POISON_BYTE).all()


def test_empty_and_degenerate_inputs():
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(2, 2)
    # no sequences at all
    lens = np.zeros(0, dtype=np.int32)
    bt = np.zeros((0, 4), dtype=np.int32)
    src = [np.zeros(orc.shard_bytes(S, m, 0, 3), dtype=np.uint8)]
    got = gpu_migrate(S, D, m, lens, bt, src, [3], [2] * 4)
    assert got["total"] == 0 and got["status"] == remp.REMP_OK
    assert all((d == POISON_BYTE).all() for d in got["dst"])
    # only zero-length sequences; destination pools of zero blocks
    lens = np.zeros(5, dtype=np.int32)
    bt = np.full((5, 4), -1, dtype=np.int32)
    got = gpu_migrate(S, D, m, lens, bt, src, [3], [0] * 4)
    assert got["total"] == 0 and got["status"] == remp.REMP_OK and (got["dst_bt"] == -1).all()
    # one token
    lens = np.array([0, 1, 0], dtype=np.int32)
    bt = np.array([[-1], [2], [-1]], dtype=np.int32)
    rng = np.random.default_rng(0)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, 0, 3), dtype=np.uint8)]
    want = oracle_run(S, D, m, lens, bt, src, [3], [1] * 4)
    got = gpu_migrate(S, D, m, lens, bt, src, [3], [1] * 4)
    assert_same(got, *want[:3])


def test_many_sequences_scan_spans_tiles():
    """More sequences than one scan tile (1024), ragged tail, lengths incl. zeros."""
    m = Shape(1, 1, 16, 1, 1)                      # 16-byte blocks: the tables dominate
    rng = np.random.default_rng(3)
    n = 5000 + 37
    lens = rng.integers(0, 9, size=n).astype(np.int32)
    need = lens.astype(np.int64)
    total = int(need.sum())
    pool = total + 11
    perm = rng.permutation(pool)[:total].astype(np.int32)
    bt = np.full((n, 8), -1, dtype=np.int32)
    pos = 0
    for s in range(n):
        bt[s, :need[s]] = perm[pos:pos + need[s]]; pos += need[s]
    S, D = Topo(1, 1), Topo(1, 1)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, 0, pool), dtype=np.uint8)]
    want = oracle_run(S, D, m, lens, bt, src, [pool], [total + 4], base=4)
    got = gpu_migrate(S, D, m, lens, bt, src, [pool], [total + 4], base=4)
    assert_same(got, *want[:3])


def test_capacity_error_writes_nothing():
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 6, 60, seed=1)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    src = [np.random.default_rng(0).integers(0, 256, size=orc.shard_bytes(S, m, 0, pool), dtype=np.uint8)]
    with pytest.raises(orc.CapacityError):
        orc.alloc(lens, bt.shape[1], m.block_size, 0, [total, total - 1])
    with pytest.raises(remp.RempError) as ei:
        gpu_migrate(S, D, m, lens, bt, src, [pool], [total, total - 1])
    assert ei.value.status == remp.REMP_ERR_CAPACITY
    # asynchronous flavour: no host read-back at allocation; the migration must copy nothing
    got = gpu_migrate(S, D, m, lens, bt, src, [pool], [total, total - 1], want_total=False)
    assert got["status"] == remp.REMP_ERR_CAPACITY
    assert all((d == POISON_BYTE).all() for d in got["dst"]) and (got["dst_bt"] == -7).all()
    # base offset pushes it over
    with pytest.raises(remp.RempError):
        gpu_migrate(S, D, m, lens, bt, src, [pool], [total, total], base=1)


def test_bad_block_ids_flagged_and_skipped():
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens = np.array([40, 20], dtype=np.int32)
    bt = np.array([[1, 99, 0], [-5, 2, -1]], dtype=np.int32)      # 99 out of pool, -5 negative
    src = [np.random.default_rng(0).integers(0, 256, size=orc.shard_bytes(S, m, 0, 3), dtype=np.uint8)]
    want_dst, want_dbt, want_total, rc = oracle_run(S, D, m, lens, bt, src, [3], [6, 6])
    assert rc == -6
    got = gpu_migrate(S, D, m, lens, bt, src, [3], [6, 6], want_total=False)
    assert got["status"] == remp.REMP_ERR_BAD_BLOCK_ID
    assert np.array_equal(got["dst_bt"], want_dbt)
    for a, b in zip(got["dst"], want_dst):
        assert np.array_equal(a, b)
    # a length that needs more blocks than the row has
    with pytest.raises(remp.RempError) as ei:
        gpu_migrate(S, D, m, np.array([100, 1], dtype=np.int32), bt, src, [3], [9, 9])
    assert ei.value.status == remp.REMP_ERR_BAD_LENGTH
    with pytest.raises(remp.RempError) as ei:
        gpu_migrate(S, D, m, np.array([-1, 1], dtype=np.int32), bt, src, [3], [9, 9])
    assert ei.value.status == remp.REMP_ERR_BAD_LENGTH


def test_alias_state_and_argument_errors():
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(1, 1)
    lens, bt, pool = small_workload(m, 3, 40, seed=2)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    nbytes = remp.remp_shard_bytes(S, m, 0, pool)
    buf = torch.zeros(2 * nbytes, dtype=torch.uint8, device="cuda")
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    src = remp.make_shards([buf[:nbytes]], [pool])
    with pytest.raises(remp.RempError) as ei:
        remp.remp_migrate_kv(plan, src, remp.make_shards([buf[nbytes:]], [pool]))
    assert ei.value.status == remp.REMP_ERR_STATE
    d_dbt = torch.empty_like(d_bt)
    remp.remp_alloc_dst_blocks(plan, [pool], 0, d_dbt)
    with pytest.raises(remp.RempError) as ei:
        remp.remp_migrate_kv(plan, src, remp.make_shards([buf[nbytes // 2: nbytes // 2 + nbytes]], [pool]))
    assert ei.value.status == remp.REMP_ERR_ALIAS
    with pytest.raises(remp.RempError) as ei:
        remp.remp_migrate_kv(plan, src, remp.make_shards([buf[nbytes:]], [pool - 1]))      # smaller than promised
    assert ei.value.status == remp.REMP_ERR_INVALID_ARG
    with pytest.raises(remp.RempError) as ei:
        remp.remp_migrate_kv(plan, src, remp.make_shards([buf[nbytes + 8:]], [pool - 1]))  # misaligned base
    assert ei.value.status in (remp.REMP_ERR_SHAPE, remp.REMP_ERR_INVALID_ARG)
    remp.remp_migrate_kv(plan, src, remp.make_shards([buf[nbytes:]], [pool]))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)


def test_in_place_table_rewrite_and_plan_reuse():
    """dst_block_tables may alias the source tables; a plan can be allocated and migrated twice."""
    m = Shape(2, 4, 64, 16, 2)
    S, D = Topo(2, 1), Topo(1, 2)
    lens, bt, pool = small_workload(m, 9, 70, seed=4)
    G = H.random_global(m, pool, 3)
    src = H.shards_from_global(S, m, G)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    want = oracle_run(S, D, m, lens, bt, src, [pool] * 2, [total] * 2)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    for rnd in range(2):
        d_dst = [torch.full((remp.remp_shard_bytes(D, m, r, total),), POISON_BYTE, dtype=torch.uint8, device="cuda")
                 for r in range(2)]
        d_out = torch.empty_like(d_bt)
        assert remp.remp_alloc_dst_blocks(plan, [total] * 2, 0, d_out) == total
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * 2), remp.make_shards(d_dst, [total] * 2))
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        for r in range(2):
            assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r])
        assert np.array_equal(d_out.cpu().numpy(), want[1])
    remp.remp_plan_destroy(plan)
    # in place: after the call the source table tensor holds the destination ids
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    assert remp.remp_alloc_dst_blocks(plan, [total] * 2, 0, d_bt) == total
    assert np.array_equal(d_bt.cpu().numpy(), want[1])
    remp.remp_plan_destroy(plan)


@pytest.mark.parametrize("S,D,window", [
    (Topo(2, 2), Topo(4, 1), 1),
    (Topo(4, 1), Topo(1, 3), 2),                  # windows must stop at the destination stage boundaries (3,5,7)
    (Topo(2, 3, (0, 1, 5, 7)), Topo(8, 1), 0),    # uneven source stages, 2x replication, automatic window
    (Topo(8, 2), Topo(2, 7), 3),                  # replicated source, one layer per destination stage
])
def test_host_resident_cache_streams_through_windows(S, D, window):
    m = Shape(7, 4, 64, 16, 2)
    lens, bt, pool = small_workload(m, 20, 200, seed=13, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(1)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 4 + (r % 3) for r in range(nd)]
    want_dst, want_dbt, want_total, rc = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=2)
    assert rc == 0
    got = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    src_copy = [b.copy() for b in src]
    dbt, tot, up, down = remp.remp_reshard_host(S, D, m, lens, bt, src, [pool] * ns, got, dst_nb, base_block=2,
                                                window_layers=window)
    assert tot == want_total and np.array_equal(dbt, want_dbt)
    for r in range(nd):
        assert np.array_equal(got[r], want_dst[r]), r
    for a, b in zip(src, src_copy):
        assert np.array_equal(a, b)
    hs = m.block_size * m.head_dim * m.elem_bytes
    assert down == total * m.num_layers * 2 * m.num_kv_heads * orc.rep(D, m.num_kv_heads) * hs + bt.size * 4 + 8
    canonical = [r for r in range(ns) if (r % S.tp) % orc.rep(S, m.num_kv_heads) == 0]
    assert up == sum(src[r].size for r in canonical) + lens.size * 4 + bt.size * 4


def test_host_resident_capacity_error_leaves_destination_untouched():
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 6, 60, seed=1)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    src = [np.zeros(orc.shard_bytes(S, m, 0, pool), dtype=np.uint8)]
    got = H.poison_like([orc.shard_bytes(D, m, r, total - 1) for r in range(2)])
    with pytest.raises(remp.RempError) as ei:
        remp.remp_reshard_host(S, D, m, lens, bt, src, [pool], got, [total - 1] * 2)
    assert ei.value.status == remp.REMP_ERR_CAPACITY
    assert all((g == POISON_BYTE).all() for g in got)


@pytest.mark.parametrize("S,D,window", [
    (Topo(2, 2), Topo(4, 1), 1),
    (Topo(4, 1), Topo(1, 3), 2),                  # windows straddle destination stage boundaries (3,5,7)
    (Topo(2, 3, (0, 1, 5, 7)), Topo(8, 1), 3),    # uneven source stages, replication
    (Topo(1, 7), Topo(2, 1), 7),                  # one window = everything
])
def test_layer_windows_with_per_layer_allocations(S, D, window):
    """Layer-wise streaming: every (rank, window) lives in its own allocation; windows run in shuffled
    order; the union equals one whole-cache migration (checked against the oracle)."""
    m = Shape(7, 4, 64, 16, 2)
    L = m.num_layers
    lens, bt, pool = small_workload(m, 16, 150, seed=17, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(5)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 2 + (r % 2) for r in range(nd)]
    want_dst, want_dbt, want_total, rc = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=1)
    assert rc == 0
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    assert remp.remp_alloc_dst_blocks(plan, dst_nb, 1, d_dbt) == want_total
    windows = [(lo, min(L, lo + window)) for lo in range(0, L, window)]
    order = rng.permutation(len(windows))
    got = [np.full_like(w, POISON_BYTE) for w in want_dst]

    def in_window(T, r, lo, hi):
        p = r // T.tp
        a, b = max(lo, orc.stage_first(T, L, p)), min(hi, orc.stage_first(T, L, p + 1))
        return (a - orc.stage_first(T, L, p), b - orc.stage_first(T, L, p)) if b > a else None

    empty = torch.empty(0, dtype=torch.uint8, device="cuda")
    for wi in order:
        lo, hi = windows[wi]
        s_bufs, d_bufs, d_rng = [], [], []
        for r in range(ns):
            w_ = in_window(S, r, lo, hi)
            lb = orc.layer_slab_bytes(S, m, pool)
            s_bufs.append(to_dev(src[r][w_[0] * lb:w_[1] * lb].copy()) if w_ else empty)
        for r in range(nd):
            w_ = in_window(D, r, lo, hi)
            lb = orc.layer_slab_bytes(D, m, dst_nb[r])
            d_bufs.append(torch.full(((w_[1] - w_[0]) * lb,), POISON_BYTE, dtype=torch.uint8, device="cuda") if w_ else empty)
            d_rng.append((w_[0] * lb, w_[1] * lb) if w_ else None)
        remp.remp_migrate_kv_layers(plan, lo, hi, remp.make_shards(s_bufs, [pool] * ns), remp.make_shards(d_bufs, dst_nb))
        torch.cuda.synchronize()
        for r in range(nd):
            if d_rng[r]:
                got[r][d_rng[r][0]:d_rng[r][1]] = d_bufs[r].cpu().numpy()
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    for r in range(nd):
        assert np.array_equal(got[r], want_dst[r]), r


@pytest.mark.parametrize("fraction", [0.0, 0.3, 0.7, 1.0, 1.5])
def test_capacity_constrained_allocation_preempts_the_tail(fraction):
    """Section 3.4.5 capacity constraint: the destination holds only part of the live footprint; the longest
    prefix of sequences that fits is migrated, the rest is preempted. Tables, mask, counts and every
    destination byte equal the oracle's."""
    m = Shape(3, 4, 64, 16, 2)
    S, D = Topo(2, 1), Topo(4, 3)
    lens, bt, pool = small_workload(m, 1500, 120, seed=23, zero_fraction=0.05)       # spans two scan tiles
    ns, nd = S.tp * S.pp, D.tp * D.pp
    need = -(-lens.astype(np.int64) // m.block_size)
    cap = int(fraction * need.sum())
    base = 2
    dst_nb = [base + cap + (r % 3) for r in range(nd)]
    rng = np.random.default_rng(3)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    want_dbt, want_pre, want_total = orc.alloc_preempt(lens, bt.shape[1], m.block_size, base, dst_nb)
    kept_lens = np.where(want_pre == 0, lens, 0).astype(np.int32)
    want_dst = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, kept_lens, bt, want_dbt, src, [pool] * ns, want_dst, dst_nb, nthreads=4) == 0
    if fraction >= 1.0:
        assert want_pre.sum() == 0
    if fraction == 0.0:
        assert want_total == 0

    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want_dst]
    d_dbt = torch.full_like(d_bt, -7)
    d_pre = torch.full((len(lens),), -7, dtype=torch.int32, device="cuda")
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    total, npre = remp.remp_alloc_dst_blocks_preempt(plan, dst_nb, base, d_dbt, d_pre)
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns), remp.make_shards(d_dst, dst_nb))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    assert total == want_total and npre == int(want_pre.sum())
    assert np.array_equal(d_pre.cpu().numpy(), want_pre)
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    for r in range(nd):
        assert np.array_equal(d_dst[r].cpu().numpy(), want_dst[r]), r


def _layout_strides(T, m, layout):
    de = m.head_dim * m.elem_bytes
    hl = orc.heads_per_rank(T, m.num_kv_heads)
    return {"head": de, "token": hl * de} if layout == "token" else {}


@pytest.mark.parametrize("src_layout,dst_layout", [("token", "token"), ("token", "head"), ("head", "token")])
@pytest.mark.parametrize("shape,S,D", [
    (Shape(3, 8, 128, 16, 2), Topo(4, 1), Topo(8, 1)),       # 70B-like split, 256-byte rows
    (Shape(3, 8, 128, 16, 2), Topo(8, 1), Topo(2, 3)),       # merge 4 sources per destination block
    (Shape(3, 8, 128, 16, 2), Topo(2, 1), Topo(2, 3)),       # TP unchanged: whole token-major blocks are contiguous
    (Shape(2, 4, 128, 32, 1), Topo(2, 1), Topo(8, 2)),       # fp8-sized elements, replication
    (Shape(2, 6, 40, 8, 2), Topo(3, 1), Topo(2, 1)),         # 80-byte rows (5 vectors), non-nesting head ranges
    (Shape(2, 2, 512, 16, 4), Topo(1, 1), Topo(2, 2)),       # 2 KiB rows
    (Shape(3, 8, 64, 16, 1), Topo(4, 1), Topo(8, 1)),        # head_dim 64 x 1 byte: 64-byte rows cut out of 128-byte rows
    (Shape(3, 8, 128, 1, 2), Topo(4, 1), Topo(8, 1)),        # block_size 1: a block is a single token row
    (Shape(3, 4, 16, 4, 1), Topo(1, 1), Topo(4, 1)),         # 16-byte rows: runs of 64 bytes, several blocks per item
    (Shape(3, 8, 64, 8, 1), Topo(4, 1), Topo(8, 1)),         # 512-byte strided runs: groups of 8 blocks
    (Shape(3, 8, 64, 16, 1), Topo(8, 1), Topo(4, 1)),        # 1 KiB strided runs merged into 128-byte rows: groups of 4
    (Shape(2, 6, 64, 4, 1), Topo(1, 1), Topo(2, 1)),         # 768-byte runs of 192-byte rows: groups of 5 blocks
    (Shape(2, 8, 96, 16, 2), Topo(1, 1), Topo(2, 1)),        # 768-byte rows, 16 per run: four items of 4 rows each
    (Shape(2, 4, 80, 64, 1), Topo(4, 1), Topo(1, 1)),        # 80-byte rows, 64 per run: two items of 32 rows each
    (Shape(2, 4, 80, 24, 1), Topo(2, 1), Topo(4, 1)),        # 24 rows of 80 bytes: one item of 1920 bytes
])
def test_token_major_layouts(shape, S, D, src_layout, dst_layout):
    """Blocks kept as [token][head][dim] on either side (strided rows instead of contiguous head slices)."""
    m = shape
    lens, bt, pool = small_workload(m, 30, 200, seed=41, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(2)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 3] * nd
    want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, 1, dst_nb)
    want = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, lens, bt, want_dbt, src, [pool] * ns, want, dst_nb, nthreads=4,
                       src_layout=src_layout, dst_layout=dst_layout) == 0
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want]
    d_dbt = torch.empty_like(d_bt)
    for opts in ({}, {remp.REMP_OPT_SCHEDULE: 1}):
        for t_ in d_dst:
            t_.fill_(POISON_BYTE)
        plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
        for k_, v_ in opts.items():
            remp.remp_plan_set_option(plan, k_, v_)
        assert remp.remp_alloc_dst_blocks(plan, dst_nb, 1, d_dbt) == want_total
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns, [_layout_strides(S, m, src_layout)] * ns),
                             remp.make_shards(d_dst, dst_nb, [_layout_strides(D, m, dst_layout)] * nd))
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        remp.remp_plan_destroy(plan)
        for r in range(nd):
            assert np.array_equal(d_dst[r].cpu().numpy(), want[r]), (r, opts)


def test_padded_head_stride_long_rows():
    """Head-major blocks whose head slices (8 KiB) sit 8 KiB + 256 B apart: rows longer than one 4 KiB piece."""
    m = Shape(2, 4, 128, 32, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 10, 300, seed=43)
    hs = m.block_size * m.head_dim * m.elem_bytes
    pad = 256
    rng = np.random.default_rng(6)
    dense = [rng.integers(0, 256, size=orc.shard_bytes(S, m, 0, pool), dtype=np.uint8)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total] * 2
    want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, 0, dst_nb)
    want = H.poison_like([orc.shard_bytes(D, m, r, total) for r in range(2)])
    assert orc.migrate(S, D, m, lens, bt, want_dbt, dense, [pool], want, dst_nb) == 0
    # embed the dense source [l][2][nb][4 heads][hs] into a padded-head buffer
    v = dense[0].reshape(2, 2, pool, 4, hs)
    padded = np.full((2, 2, pool, 4, hs + pad), 0x11, dtype=np.uint8)
    padded[..., :hs] = v
    d_src = [to_dev(padded.reshape(-1))]
    sstr = [{"head": hs + pad, "block": 4 * (hs + pad)}]
    d_dst = [torch.full((2 * 2 * total * 2 * (hs + pad),), POISON_BYTE, dtype=torch.uint8, device="cuda") for _ in range(2)]
    dstr = [{"head": hs + pad, "block": 2 * (hs + pad)}] * 2
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    assert remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt) == want_total
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool], sstr), remp.make_shards(d_dst, dst_nb, dstr))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    for r in range(2):
        got = d_dst[r].cpu().numpy().reshape(2, 2, total, 2, hs + pad)
        assert np.array_equal(got[..., :hs].reshape(-1), want[r])
        assert (got[..., hs:] == POISON_BYTE).all()


def _shared_tables(rng, n, bs, pool, max_len, share):
    lens = rng.integers(0, max_len + 1, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // bs)
    maxb = int(need.max(initial=1)) + 1
    bt = np.full((n, maxb), -1, dtype=np.int32)
    free = list(rng.permutation(pool))
    for s in range(n):
        k = 0
        if s and rng.random() < share:
            o = int(rng.integers(0, s))
            k = int(rng.integers(0, min(need[s], need[o]) + 1))
            bt[s, :k] = bt[o, :k]
        for j in range(k, need[s]):
            bt[s, j] = free.pop()
    return lens, bt


@pytest.mark.parametrize("share", [0.0, 0.5, 0.95])
def test_shared_prefix_blocks_stay_shared_and_are_copied_once(share):
    """Section 3.4.5 (prefixes): equal source blocks get one destination block; ids, tables, the number of
    distinct blocks and every destination byte equal the oracle's."""
    m = Shape(3, 4, 64, 16, 2)
    S, D = Topo(2, 1), Topo(4, 3)
    rng = np.random.default_rng(int(share * 100) + 1)
    pool = 60000
    lens, bt = _shared_tables(rng, 1300, m.block_size, pool, 500, share)       # > 1024 entries per scan tile
    ns, nd = S.tp * S.pp, D.tp * D.pp
    want_dbt, want_total, bad = orc.alloc_shared(lens, bt, m.block_size, 3, pool, [10**7] * nd)
    assert not bad
    entries = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    assert (want_total < entries) == (share > 0)
    dst_nb = [3 + want_total + (r % 2) for r in range(nd)]
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    want_dst = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, lens, bt, want_dbt, src, [pool] * ns, want_dst, dst_nb, nthreads=4) == 0

    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want_dst]
    d_dbt = torch.full_like(d_bt, -7)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    launches0 = remp.remp_kernel_launch_count()
    total = remp.remp_alloc_dst_blocks_shared(plan, dst_nb, 3, pool, d_dbt)
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns), remp.make_shards(d_dst, dst_nb))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    assert remp.remp_kernel_launch_count() - launches0 == 5
    remp.remp_plan_destroy(plan)
    assert total == want_total
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    for r in range(nd):
        assert np.array_equal(d_dst[r].cpu().numpy(), want_dst[r]), r
    # capacity is judged on distinct blocks
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    if want_total > 0:
        with pytest.raises(remp.RempError) as ei:
            remp.remp_alloc_dst_blocks_shared(plan, [3 + want_total - 1] * nd, 3, pool, d_dbt)
        assert ei.value.status == remp.REMP_ERR_CAPACITY
    remp.remp_plan_destroy(plan)


def test_shared_allocation_reports_ids_outside_the_pool():
    m = Shape(1, 1, 64, 16, 2)
    T = Topo(1, 1)
    lens = np.array([32, 32], dtype=np.int32)
    bt = np.array([[3, 50], [3, -4]], dtype=np.int32)
    want_dbt, want_total, bad = orc.alloc_shared(lens, bt, 16, 0, 10, [9])
    assert bad and want_total == 3
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(T, T, m, d_lens, d_bt)
    with pytest.raises(remp.RempError) as ei:
        remp.remp_alloc_dst_blocks_shared(plan, [9], 0, 10, d_dbt)
    assert ei.value.status == remp.REMP_ERR_BAD_BLOCK_ID
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    remp.remp_plan_destroy(plan)


def test_host_resident_direct_path_with_page_locked_buffers():
    """Page-locked, device-mapped host buffers: the kernel reads and writes host memory itself (window 0);
    the same buffers through the staged path (window 2) must give the same bytes and the oracle's."""
    m = Shape(6, 4, 64, 16, 2)
    S, D = Topo(2, 2), Topo(8, 1)
    lens, bt, pool = small_workload(m, 20, 200, seed=19, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(4)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 2] * nd
    want_dst, want_dbt, want_total, rc = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=1)
    assert rc == 0
    p_src = [torch.from_numpy(b).pin_memory() for b in src]
    hs = m.block_size * m.head_dim * m.elem_bytes
    live_bytes = total * m.num_layers * 2 * m.num_kv_heads * hs
    for window in (0, 2):
        p_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8).pin_memory() for b in want_dst]
        dbt, tot, up, down = remp.remp_reshard_host(S, D, m, lens, bt, p_src, [pool] * ns, p_dst, dst_nb,
                                                    base_block=1, window_layers=window)
        assert tot == want_total and np.array_equal(dbt, want_dbt)
        for r in range(nd):
            assert np.array_equal(p_dst[r].numpy(), want_dst[r]), (window, r)
        assert down == 2 * live_bytes + bt.size * 4 + 8            # 2x replication on the destination side
        if window == 0:                                             # pool 1.25x the live blocks: direct path
            assert up == live_bytes + lens.size * 4 + bt.size * 4   # only live blocks were read
    for a, b in zip(p_src, src):
        assert np.array_equal(a.numpy(), b)


@pytest.mark.parametrize("src_layout,dst_layout", [("head", "head"), ("token", "token"), ("token", "head"), ("head", "token")])
@pytest.mark.parametrize("shape,S,D", [
    (Shape(3, 8, 128, 16, 2), Topo(4, 1), Topo(8, 1)),       # 4 KiB runs
    (Shape(3, 8, 128, 16, 2), Topo(8, 1), Topo(2, 3)),
    (Shape(2, 8, 128, 32, 1), Topo(2, 1), Topo(16, 1)),      # fp8-sized, replication, many partial blocks
    (Shape(3, 4, 64, 16, 2), Topo(1, 1), Topo(2, 1)),        # 2-head runs (head slices inside a chunk)
    (Shape(2, 2, 64, 128, 2), Topo(1, 2), Topo(1, 1)),       # whole blocks, 16 KiB head slices (several chunks)
    (Shape(3, 8, 64, 8, 1), Topo(4, 1), Topo(8, 1)),         # 512-byte runs: groups of blocks, partial last block
    (Shape(2, 6, 64, 4, 1), Topo(1, 1), Topo(2, 1)),         # 768-byte runs: groups of 5 blocks
])
def test_valid_tokens_only(shape, S, D, src_layout, dst_layout):
    """REMP_OPT_VALID_TOKENS_ONLY: slack token slots of partial blocks are neither read nor written."""
    m = shape
    lens, bt, pool = small_workload(m, 60, 3 * m.block_size - 1, seed=61, zero_fraction=0.1)   # mostly partial blocks
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(8)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 1] * nd
    want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, 0, dst_nb)
    want = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, lens, bt, want_dbt, src, [pool] * ns, want, dst_nb, nthreads=4, src_layout=src_layout,
                       dst_layout=dst_layout, valid_only=True) == 0
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dbt = torch.empty_like(d_bt)
    for extra in ({}, {remp.REMP_OPT_SCHEDULE: 1}, {remp.REMP_OPT_KERNEL: 2}, {remp.REMP_OPT_VEC_BYTES: 32}):
        d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want]
        plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
        remp.remp_plan_set_option(plan, remp.REMP_OPT_VALID_TOKENS_ONLY, 1)
        for k_, v_ in extra.items():
            remp.remp_plan_set_option(plan, k_, v_)
        assert remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt) == want_total
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns, [_layout_strides(S, m, src_layout)] * ns),
                             remp.make_shards(d_dst, dst_nb, [_layout_strides(D, m, dst_layout)] * nd))
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        r_, w_ = remp.remp_plan_traffic_tokens(plan, int(lens.sum()))
        remp.remp_plan_destroy(plan)
        for r in range(nd):
            assert np.array_equal(d_dst[r].cpu().numpy(), want[r]), (r, extra)
        written = sum(int((t_ != POISON_BYTE).sum().item()) for t_ in d_dst)
        assert 0.97 * w_ <= written <= w_                          # only bytes of tokens in use were written


def test_two_plans_on_two_streams_run_concurrently():
    """Independent plans on independent streams share only the library's pool: results stay exact."""
    m = Shape(4, 8, 128, 16, 2)
    cases = []
    for i, (S, D) in enumerate(((Topo(4, 1), Topo(8, 1)), (Topo(2, 2), Topo(1, 4)))):
        lens, bt, pool = small_workload(m, 300, 400, seed=70 + i)
        ns, nd = S.tp * S.pp, D.tp * D.pp
        rng = np.random.default_rng(i)
        src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
        total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
        dst_nb = [total] * nd
        want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb)
        cases.append((S, D, lens, bt, pool, src, dst_nb, want))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    state = []
    for (S, D, lens, bt, pool, src, dst_nb, want), st in zip(cases, streams):
        with torch.cuda.stream(st):
            d_lens, d_bt = to_dev(lens), to_dev(bt)
            d_src = [to_dev(b) for b in src]
            d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want[0]]
            d_dbt = torch.empty_like(d_bt)
        state.append((d_lens, d_bt, d_src, d_dst, d_dbt))
    torch.cuda.synchronize()
    plans = []
    for rep_ in range(3):                       # interleave enqueues of both plans, several times
        for (S, D, lens, bt, pool, src, dst_nb, want), st, (d_lens, d_bt, d_src, d_dst, d_dbt) in zip(cases, streams, state):
            plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
            remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt, want_total=False, stream=st)
            remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * len(d_src)), remp.make_shards(d_dst, dst_nb), stream=st)
            plans.append((plan, st))
    for plan, st in plans:
        assert remp.remp_plan_status(plan, st) == remp.REMP_OK
        remp.remp_plan_destroy(plan)
    torch.cuda.synchronize()
    for (S, D, lens, bt, pool, src, dst_nb, want), (d_lens, d_bt, d_src, d_dst, d_dbt) in zip(cases, state):
        assert np.array_equal(d_dbt.cpu().numpy(), want[1])
        for r in range(len(d_dst)):
            assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r])
    remp.remp_release_cached_memory()


def test_many_short_sequences_at_scale():
    """200k sequences: the scan walks ~200 tiles, the remapper strides its grid, the shared allocator scans
    300k entries - all equal to the oracle."""
    m = Shape(1, 1, 16, 4, 1)
    rng = np.random.default_rng(11)
    n = 200_003
    lens = rng.integers(0, 9, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // 4)
    total = int(need.sum())
    pool = total + 100
    ids = rng.permutation(pool)[:total].astype(np.int32)
    bt = np.full((n, 2), -1, dtype=np.int32)
    pos = np.concatenate([[0], np.cumsum(need)])
    for j in range(2):
        sel = need > j
        bt[sel, j] = ids[pos[:-1][sel] + j]
    a_, b_ = np.arange(4, n - 1, 7), np.arange(5, n, 7)        # some shared first blocks
    k_ = min(len(a_), len(b_))
    both = (need[a_[:k_]] > 0) & (need[b_[:k_]] > 0)
    bt[b_[:k_][both], 0] = bt[a_[:k_][both], 0]
    T = Topo(1, 1)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(T, T, m, d_lens, d_bt)
    want_dbt, _off, want_total = orc.alloc(lens, 2, 4, 5, [10**7])
    assert remp.remp_alloc_dst_blocks(plan, [10**7], 5, d_dbt) == want_total
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    want_dbt, want_pre, want_total = orc.alloc_preempt(lens, 2, 4, 5, [5 + total // 3])
    d_pre = torch.empty(n, dtype=torch.int32, device="cuda")
    tot, npre = remp.remp_alloc_dst_blocks_preempt(plan, [5 + total // 3], 5, d_dbt, d_pre)
    assert tot == want_total and npre == int(want_pre.sum())
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt) and np.array_equal(d_pre.cpu().numpy(), want_pre)
    want_dbt, want_total, bad = orc.alloc_shared(lens, bt, 4, 5, pool, [10**7])
    assert not bad
    assert remp.remp_alloc_dst_blocks_shared(plan, [10**7], 5, pool, d_dbt) == want_total
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    remp.remp_plan_destroy(plan)


def test_source_in_page_locked_host_memory_destination_on_device():
    """A swapped-out cache (page-locked host memory) is re-sharded straight into device pools by remp_migrate_kv."""
    m = Shape(4, 8, 128, 16, 2)
    S, D = Topo(4, 1), Topo(2, 2)
    lens, bt, pool = small_workload(m, 40, 300, seed=81)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(9)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total] * nd
    want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb)
    h_src = [torch.from_numpy(b).pin_memory() for b in src]
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want[0]]
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    assert remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt) == want[2]
    # make_shards marshals data_ptr(): for pinned tensors that is a host address the device can use directly
    remp.remp_migrate_kv(plan, remp.make_shards(h_src, [pool] * ns), remp.make_shards(d_dst, dst_nb))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    for r in range(nd):
        assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r])


def test_round_trip_from_a_compact_table_reproduces_the_input_bytes_on_the_gpu():
    m = Shape(4, 8, 128, 16, 2)
    lens = np.array([300, 0, 64, 1000, 1, 17], dtype=np.int32)
    need = -(-lens.astype(np.int64) // m.block_size)
    total = int(need.sum())
    bt, _off, _t = orc.alloc(lens, int(need.max()) + 1, m.block_size, 0, [total])
    A, B = Topo(4, 2), Topo(8, 1)
    rng = np.random.default_rng(21)
    src = [rng.integers(0, 256, size=orc.shard_bytes(A, m, r, total), dtype=np.uint8) for r in range(8)]
    mid = gpu_migrate(A, B, m, lens, bt, src, [total] * 8, [total] * 8)
    assert np.array_equal(mid["dst_bt"], bt)
    back = gpu_migrate(B, A, m, lens, mid["dst_bt"], mid["dst"], [total] * 8, [total] * 8)
    for a, b in zip(src, back["dst"]):
        assert a.tobytes() == b.tobytes()


@pytest.mark.parametrize("n", [8192, 8193, 9217, 20000])
def test_demand_scan_single_and_multi_cta_paths_agree_with_the_oracle(n):
    """Around the switch from the one-CTA scan to the three-launch scan: ids, totals, preemption masks,
    capacity and bad-length reporting are those of the oracle's serial sum."""
    m = Shape(1, 1, 16, 4, 1)
    rng = np.random.default_rng(n)
    lens = rng.integers(0, 13, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // 4)
    total = int(need.sum())
    bt = np.zeros((n, 3), dtype=np.int32)
    T = Topo(1, 1)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    plan = remp.remp_plan_create(T, T, m, d_lens, d_bt)
    want_dbt, _off, want_total = orc.alloc(lens, 3, 4, 7, [7 + total])
    assert remp.remp_alloc_dst_blocks(plan, [7 + total], 7, d_dbt) == want_total
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
    with pytest.raises(remp.RempError) as ei:
        remp.remp_alloc_dst_blocks(plan, [7 + total - 1], 7, d_dbt)
    assert ei.value.status == remp.REMP_ERR_CAPACITY
    d_pre = torch.empty(n, dtype=torch.int32, device="cuda")
    for cap in (0, total // 2, total - 1, total, total + 5):
        want_dbt, want_pre, want_tot = orc.alloc_preempt(lens, 3, 4, 7, [7 + cap])
        tot, npre = remp.remp_alloc_dst_blocks_preempt(plan, [7 + cap], 7, d_dbt, d_pre)
        assert (tot, npre) == (want_tot, int(want_pre.sum()))
        assert np.array_equal(d_dbt.cpu().numpy(), want_dbt) and np.array_equal(d_pre.cpu().numpy(), want_pre)
    remp.remp_plan_destroy(plan)
    bad = lens.copy()
    bad[n - 3] = 100                                    # needs 25 blocks, the row has 3
    d_bad = to_dev(bad)
    plan = remp.remp_plan_create(T, T, m, d_bad, d_bt)
    with pytest.raises(remp.RempError) as ei:
        remp.remp_alloc_dst_blocks(plan, [10**7], 0, d_dbt)
    assert ei.value.status == remp.REMP_ERR_BAD_LENGTH
    remp.remp_plan_destroy(plan)


@pytest.mark.parametrize("shape,S,D", [
    (Shape(2, 4, 8, 16, 1), Topo(1, 1), Topo(2, 1)),      # 8-byte token rows, 128-byte head slices (several blocks per item)
    (Shape(2, 4, 8, 16, 1), Topo(4, 1), Topo(1, 2)),
    (Shape(2, 4, 24, 32, 1), Topo(1, 1), Topo(2, 1)),     # 24-byte token rows, 768-byte slices, 2-head runs
    (Shape(2, 4, 24, 32, 1), Topo(2, 1), Topo(8, 1)),     # ... with 2x replication
    (Shape(3, 8, 40, 16, 1), Topo(2, 1), Topo(4, 1)),     # 40-byte token rows, 640-byte slices
    (Shape(2, 2, 8, 64, 2), Topo(1, 1), Topo(2, 1)),      # 16-byte token rows, 1 KiB slices (32-byte vectors asked for)
    (Shape(2, 2, 12, 512, 1), Topo(1, 2), Topo(2, 1)),    # 12-byte token rows, 6 KiB slices: several chunks per run
])
@pytest.mark.parametrize("padded", [False, True])
def test_valid_tokens_only_with_token_rows_narrower_than_a_vector(shape, S, D, padded):
    """A 16-byte vector may start inside the last token in use and end in the first slack token: the slack
    bytes must still keep the destination's bytes (valid-tokens-only mode copies that vector byte by byte)."""
    m = shape
    lens, bt, pool = small_workload(m, 50, 3 * m.block_size - 1, seed=67, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(9)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 2] * nd
    want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, 1, dst_nb)
    want = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, lens, bt, want_dbt, src, [pool] * ns, want, dst_nb, nthreads=4, valid_only=True) == 0
    hs = m.block_size * m.head_dim * m.elem_bytes
    pad = 48 if padded else 0                   # padded head slices take the strided-row kernel
    hl_s, hl_d = orc.heads_per_rank(S, m.num_kv_heads), orc.heads_per_rank(D, m.num_kv_heads)

    def embed(flat, layers, nb, hl):
        v = flat.reshape(layers, 2, nb, hl, hs)
        out = np.full((layers, 2, nb, hl, hs + pad), 0x3C, dtype=np.uint8)
        out[..., :hs] = v
        return out.reshape(-1)

    def stage_layers(T, r):
        lo, hi = H.stage_ranges(T, m.num_layers)[r // T.tp]
        return hi - lo

    d_src = [to_dev(embed(src[r], stage_layers(S, r), pool, hl_s)) for r in range(ns)]
    sstr = [{"head": hs + pad, "block": hl_s * (hs + pad)}] * ns if padded else None
    dstr = [{"head": hs + pad, "block": hl_d * (hs + pad)}] * nd if padded else None
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    for extra in ({}, {remp.REMP_OPT_VEC_BYTES: 32}, {remp.REMP_OPT_SCHEDULE: 1}, {remp.REMP_OPT_CHUNK_BYTES: 512}):
        d_dst = [to_dev(embed(np.full(len(want[r]), POISON_BYTE, dtype=np.uint8), stage_layers(D, r), dst_nb[r], hl_d))
                 for r in range(nd)]
        plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
        remp.remp_plan_set_option(plan, remp.REMP_OPT_VALID_TOKENS_ONLY, 1)
        for k_, v_ in extra.items():
            remp.remp_plan_set_option(plan, k_, v_)
        assert remp.remp_alloc_dst_blocks(plan, dst_nb, 1, d_dbt) == want_total
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns, sstr), remp.make_shards(d_dst, dst_nb, dstr))
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        remp.remp_plan_destroy(plan)
        for r in range(nd):
            got = d_dst[r].cpu().numpy().reshape(stage_layers(D, r), 2, dst_nb[r], hl_d, hs + pad)
            assert np.array_equal(got[..., :hs].reshape(-1), want[r]), (r, extra)
            assert (got[..., hs:] == 0x3C).all()


@pytest.mark.parametrize("n,maxlen", [(1, 40), (8, 256), (31, 500), (32, 900), (33, 500), (32, 1200), (64, 3000), (1000, 900),
                                      (1024, 700)])
@pytest.mark.parametrize("preempt", [False, True])
def test_fused_and_separate_allocation_paths_agree_with_the_oracle(n, maxlen, preempt):
    """remp_alloc_dst_blocks as one cluster launch (REMP_OPT_ALLOC_PATH 1) and as separate scan and remap launches
    (2): tables, totals, preempted mask, pair-driven copies and the status all equal the oracle's."""
    m = Shape(2, 2, 16, 8, 2)
    S, D = Topo(1, 1), Topo(2, 2)
    lens, bt, pool = small_workload(m, n, maxlen, seed=71 + n, zero_fraction=0.1)
    need = -(-lens.astype(np.int64) // m.block_size)
    base = 3
    cap = int(0.6 * need.sum()) if preempt else int(need.sum())
    dst_nb = [base + cap + (r % 2) for r in range(4)]
    rng = np.random.default_rng(5)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, 0, pool), dtype=np.uint8)]
    if preempt:
        want_dbt, want_pre, want_total = orc.alloc_preempt(lens, bt.shape[1], m.block_size, base, dst_nb)
        kept_lens = np.where(want_pre == 0, lens, 0).astype(np.int32)
    else:
        want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, base, dst_nb)
        want_pre, kept_lens = np.zeros(n, np.int32), lens
    want_dst = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(4)])
    assert orc.migrate(S, D, m, kept_lens, bt, want_dbt, src, [pool], want_dst, dst_nb, nthreads=4) == 0
    d_lens, d_bt, d_src = to_dev(lens), to_dev(bt), [to_dev(src[0])]
    for path in (1, 2, 0):
        d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want_dst]
        d_dbt = torch.full_like(d_bt, -7)
        d_pre = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
        remp.remp_plan_set_option(plan, remp.REMP_OPT_ALLOC_PATH, path)
        launches0 = remp.remp_kernel_launch_count()
        if preempt:
            total, npre = remp.remp_alloc_dst_blocks_preempt(plan, dst_nb, base, d_dbt, d_pre)
            assert npre == int(want_pre.sum()) and np.array_equal(d_pre.cpu().numpy(), want_pre)
        else:
            total = remp.remp_alloc_dst_blocks(plan, dst_nb, base, d_dbt)
        assert remp.remp_kernel_launch_count() - launches0 == (2 if path == 2 else 1)
        for _ in range(2):                       # twice: the tile scheduler's counters return to zero by themselves
            remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool]), remp.make_shards(d_dst, dst_nb))
        assert remp.remp_kernel_launch_count() - launches0 == (4 if path == 2 else 3)
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        remp.remp_plan_destroy(plan)
        assert total == want_total
        assert np.array_equal(d_dbt.cpu().numpy(), want_dbt), path
        for r in range(4):
            assert np.array_equal(d_dst[r].cpu().numpy(), want_dst[r]), (path, r)


def test_fused_allocation_reports_errors_like_the_separate_launches():
    m = Shape(2, 2, 16, 8, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 40, 200, seed=3)
    need = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    d_bt = to_dev(bt)
    bad_bt = bt.copy()
    bad_bt[7, 0] = -5                                   # a live entry below zero
    for path in (1, 2):
        # capacity: nothing is written
        d_dbt = torch.full_like(d_bt, -7)
        plan = remp.remp_plan_create(S, D, m, to_dev(lens), d_bt)
        remp.remp_plan_set_option(plan, remp.REMP_OPT_ALLOC_PATH, path)
        with pytest.raises(remp.RempError) as e:
            remp.remp_alloc_dst_blocks(plan, [need - 1, need + 5], 0, d_dbt)
        assert e.value.status == remp.REMP_ERR_CAPACITY
        assert (d_dbt == -7).all()
        remp.remp_plan_destroy(plan)
        # a length wider than its row
        long_lens = lens.copy()
        long_lens[3] = (bt.shape[1] + 1) * m.block_size
        plan = remp.remp_plan_create(S, D, m, to_dev(long_lens), d_bt)
        remp.remp_plan_set_option(plan, remp.REMP_OPT_ALLOC_PATH, path)
        with pytest.raises(remp.RempError) as e:
            remp.remp_alloc_dst_blocks(plan, [need + 99] * 2, 0, d_dbt)
        assert e.value.status == remp.REMP_ERR_BAD_LENGTH
        assert (d_dbt == -7).all()
        remp.remp_plan_destroy(plan)
        # negative source id: flagged, tables still written
        plan = remp.remp_plan_create(S, D, m, to_dev(lens), to_dev(bad_bt))
        remp.remp_plan_set_option(plan, remp.REMP_OPT_ALLOC_PATH, path)
        with pytest.raises(remp.RempError) as e:
            remp.remp_alloc_dst_blocks(plan, [need] * 2, 0, d_dbt)
        assert e.value.status == remp.REMP_ERR_BAD_BLOCK_ID
        want_dbt, _o, _t = orc.alloc(lens, bt.shape[1], m.block_size, 0, [need] * 2)
        assert np.array_equal(d_dbt.cpu().numpy(), want_dbt)
        remp.remp_plan_destroy(plan)
    # outside the fused range the forced fused path is refused, the automatic choice still works
    n_big = 1025
    lens2, bt2, _pool2 = small_workload(m, n_big, 30, seed=4)
    plan = remp.remp_plan_create(S, D, m, to_dev(lens2), to_dev(bt2))
    remp.remp_plan_set_option(plan, remp.REMP_OPT_ALLOC_PATH, 1)
    with pytest.raises(remp.RempError) as e:
        remp.remp_alloc_dst_blocks(plan, [10 ** 6] * 2, 0, torch.empty_like(to_dev(bt2)))
    assert e.value.status == remp.REMP_ERR_INVALID_ARG
    remp.remp_plan_destroy(plan)


def test_more_ranks_than_the_kernel_parameters_hold():
    """128 ranks: the addressing tables exceed the kernel-parameter pool and are read from device memory."""
    m = Shape(4, 64, 16, 4, 1)                               # 64-byte head slices
    S, D = Topo(64, 1), Topo(32, 2)
    lens, bt, pool = small_workload(m, 12, 40, seed=13)
    ns, nd = 64, 64
    rng = np.random.default_rng(2)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 1] * nd
    want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb)
    assert want[3] == 0
    for opts in ({}, {remp.REMP_OPT_KERNEL: 2}, {remp.REMP_OPT_ORDER: 1}):
        got = gpu_migrate(S, D, m, lens, bt, src, [pool] * ns, dst_nb, options=opts)
        assert_same(got, *want[:3], tag=opts)
    # and with replication on both sides (2 heads: 16 ranks per head -> 32 ranks per head, two stages)
    m2 = Shape(2, 2, 16, 4, 1)
    S2, D2 = Topo(32, 1), Topo(64, 2)
    src2 = [rng.integers(0, 256, size=orc.shard_bytes(S2, m2, r, pool), dtype=np.uint8) for r in range(32)]
    want2 = oracle_run(S2, D2, m2, lens, bt, src2, [pool] * 32, [total] * 128)
    assert want2[3] == 0
    got2 = gpu_migrate(S2, D2, m2, lens, bt, src2, [pool] * 32, [total] * 128)
    assert_same(got2, *want2[:3])


def test_unsupported_chunk_size_is_refused_before_anything_runs():
    m = Shape(2, 4, 128, 16, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 6, 100, seed=1)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    d_src = [torch.zeros(orc.shard_bytes(S, m, 0, pool), dtype=torch.uint8, device="cuda")]
    d_dst = [torch.full((orc.shard_bytes(D, m, r, total),), POISON_BYTE, dtype=torch.uint8, device="cuda") for r in range(2)]
    d_bt = to_dev(bt)
    plan = remp.remp_plan_create(S, D, m, to_dev(lens), d_bt)
    remp.remp_plan_set_option(plan, remp.REMP_OPT_CHUNK_BYTES, 1536)
    remp.remp_alloc_dst_blocks(plan, [total] * 2, 0, torch.empty_like(d_bt))
    with pytest.raises(remp.RempError) as e:
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool]), remp.make_shards(d_dst, [total] * 2))
    assert e.value.status == remp.REMP_ERR_INVALID_ARG
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    assert all(bool((t == POISON_BYTE).all()) for t in d_dst)
    remp.remp_plan_set_option(plan, remp.REMP_OPT_KERNEL, 2)      # the bulk-copy ring takes any multiple of 512
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool]), remp.make_shards(d_dst, [total] * 2))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)


def test_bulk_kernel_wait_limit_is_reported_and_leaves_the_context_usable():
    """The bulk-copy kernel's bounded barrier wait, made to run out (zero polls allowed): the call reports
    REMP_ERR_CUDA with the wait-limit message, every destination block is either the oracle's or untouched,
    and the next call with the default limit is exact."""
    m = Shape(3, 8, 128, 16, 2)
    S, D = Topo(4, 1), Topo(8, 1)
    lens, bt, pool = small_workload(m, 30, 300, seed=77)
    ns, nd = 4, 8
    rng = np.random.default_rng(4)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total] * nd
    want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dbt = torch.empty_like(d_bt)
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want[0]]
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    remp.remp_plan_set_option(plan, remp.REMP_OPT_KERNEL, 2)
    remp.remp_plan_set_option(plan, remp.REMP_OPT_WAIT_SPINS, 1)          # zero polls
    remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt)
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns), remp.make_shards(d_dst, dst_nb))
    assert remp.remp_plan_status(plan) == remp.REMP_ERR_CUDA
    assert "wait limit" in remp.remp_last_error()
    hs = m.block_size * m.head_dim * m.elem_bytes
    for r in range(nd):
        got = d_dst[r].cpu().numpy().reshape(-1, hs)
        ref = want[0][r].reshape(-1, hs)
        same = (got == ref).all(axis=1)
        untouched = (got == POISON_BYTE).all(axis=1)
        assert (same | untouched).all(), r
    # same plan, default limit: exact, and the error word starts clean
    remp.remp_plan_set_option(plan, remp.REMP_OPT_WAIT_SPINS, 0)
    remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt)
    remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns), remp.make_shards(d_dst, dst_nb))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    for r in range(nd):
        assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r]), r


def test_overlapping_destinations_are_refused_on_the_device_and_the_host_path():
    """Two destination shards that share bytes, and a host destination that overlaps a host source, are
    REMP_ERR_ALIAS before anything moves (remp_migrate_kv and remp_reshard_host alike)."""
    m = Shape(2, 2, 64, 16, 2)
    S, D = Topo(1, 1), Topo(2, 1)
    lens, bt, pool = small_workload(m, 3, 40, seed=2)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    s_bytes = remp.remp_shard_bytes(S, m, 0, pool)
    d_bytes = remp.remp_shard_bytes(D, m, 0, total)
    d_src = torch.zeros(s_bytes, dtype=torch.uint8, device="cuda")
    buf = torch.full((2 * d_bytes,), POISON_BYTE, dtype=torch.uint8, device="cuda")
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    remp.remp_alloc_dst_blocks(plan, [total] * 2, 0, torch.empty_like(d_bt))
    with pytest.raises(remp.RempError) as ei:          # second destination starts inside the first
        remp.remp_migrate_kv(plan, remp.make_shards([d_src], [pool]),
                             remp.make_shards([buf[:d_bytes], buf[d_bytes - 256: 2 * d_bytes - 256]], [total] * 2))
    assert ei.value.status == remp.REMP_ERR_ALIAS
    assert bool((buf == POISON_BYTE).all())
    remp.remp_migrate_kv(plan, remp.make_shards([d_src], [pool]),
                         remp.make_shards([buf[:d_bytes], buf[d_bytes:]], [total] * 2))
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    # host path: pageable (staged windows) and page-locked (direct) buffers
    for pin in (False, True):
        host = torch.zeros(s_bytes + 2 * d_bytes, dtype=torch.uint8, pin_memory=pin)
        h_src = host[:s_bytes]
        before = host.clone()
        with pytest.raises(remp.RempError) as ei:      # destination 0 reaches into the source
            remp.remp_reshard_host(S, D, m, lens, bt, [h_src], [pool],
                                   [host[s_bytes - 512: s_bytes - 512 + d_bytes], host[s_bytes + d_bytes:]], [total] * 2)
        assert ei.value.status == remp.REMP_ERR_ALIAS
        with pytest.raises(remp.RempError) as ei:      # the two destinations overlap each other
            remp.remp_reshard_host(S, D, m, lens, bt, [h_src], [pool],
                                   [host[s_bytes: s_bytes + d_bytes], host[s_bytes + d_bytes - 512: s_bytes + 2 * d_bytes - 512]],
                                   [total] * 2)
        assert ei.value.status == remp.REMP_ERR_ALIAS
        assert torch.equal(host, before)
        out = remp.remp_reshard_host(S, D, m, lens, bt, [h_src], [pool],
                                     [host[s_bytes: s_bytes + d_bytes], host[s_bytes + d_bytes:]], [total] * 2)
        assert out[1] == total


@pytest.mark.parametrize("shape,S,D", [
    (Shape(2, 4, 64, 16, 2), Topo(1, 1), Topo(2, 2)),         # the Tiny configuration's first switch
    (Shape(4, 8, 128, 16, 2), Topo(4, 2), Topo(8, 1)),        # 70B-like split, 4 KiB runs
    (Shape(4, 8, 128, 16, 2), Topo(8, 1), Topo(2, 4)),        # merge heads, split stages
    (Shape(3, 8, 128, 32, 1), Topo(2, 1), Topo(16, 1)),       # 2x replication: the replicas of a head on different devices
    (Shape(3, 8, 128, 32, 1), Topo(16, 1), Topo(1, 3)),       # replicated source
    (Shape(5, 6, 72, 16, 4), Topo(3, 1), Topo(2, 1)),         # head ranges that do not nest
    (Shape(7, 2, 64, 8, 2), Topo(2, 3, (0, 1, 5, 7)), Topo(1, 2, (0, 6, 7))),
    (Shape(4, 4, 16, 4, 1), Topo(2, 1), Topo(4, 1)),          # 64-byte runs (several blocks per item)
])
@pytest.mark.parametrize("ndev", [1, 2, 3])
def test_exchange_over_logical_devices_on_one_gpu(shape, S, D, ndev):
    """remp_migrate_kv_exchange with the destination ranks spread over ndev logical devices that all happen to
    be this GPU (the pointers of 'remote' sources are local ones - the code path is the same): after the call
    of device q exactly the pools of q's ranks hold the oracle's bytes and every other pool is untouched; after
    all calls everything equals the oracle's single-device result."""
    m = shape
    lens, bt, pool = small_workload(m, 25, 200, seed=31, zero_fraction=0.1)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    rng = np.random.default_rng(12)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 2] * nd
    want = oracle_run(S, D, m, lens, bt, src, [pool] * ns, dst_nb, base=1)
    assert want[3] == 0
    sdev = [r % ndev for r in range(ns)]
    ddev = [(r + 1) % ndev for r in range(nd)]
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want[0]]
    d_dbt = torch.empty_like(d_bt)
    done = set()
    for q in range(ndev):
        plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)          # every device makes its own plan and tables
        assert remp.remp_alloc_dst_blocks(plan, dst_nb, 1, d_dbt) == want[2]
        recv, _send = remp.remp_plan_partition(plan, sdev, ddev, q)
        needed = set(int(s) for s in recv[:, 0])
        empty = torch.empty(0, dtype=torch.uint8, device="cuda")
        # hand over only what device q may touch: the sources it receives from and its own destination pools
        s_sh = remp.make_shards([d_src[r] if r in needed else empty for r in range(ns)],
                                [pool if r in needed else 0 for r in range(ns)])
        d_sh = remp.make_shards([d_dst[r] if ddev[r] == q else empty for r in range(nd)],
                                [dst_nb[r] if ddev[r] == q else 0 for r in range(nd)])
        remp.remp_migrate_kv_exchange(plan, sdev, ddev, q, s_sh, d_sh)
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        remp.remp_plan_destroy(plan)
        done |= {r for r in range(nd) if ddev[r] == q}
        for r in range(nd):
            got = d_dst[r].cpu().numpy()
            if r in done:
                assert np.array_equal(got, want[0][r]), (q, r)
            else:
                assert (got == POISON_BYTE).all(), (q, r)
    assert np.array_equal(d_dbt.cpu().numpy(), want[1])
    for a, b in zip(d_src, src):
        assert np.array_equal(a.cpu().numpy(), b)


def test_exchange_refuses_the_bulk_kernel_for_remote_sources_only():
    m = Shape(2, 4, 128, 16, 2)
    S, D = Topo(2, 1), Topo(4, 1)
    lens, bt, pool = small_workload(m, 5, 100, seed=1)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    rng = np.random.default_rng(1)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(2)]
    want = oracle_run(S, D, m, lens, bt, src, [pool] * 2, [total] * 4)
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want[0]]
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    remp.remp_plan_set_option(plan, remp.REMP_OPT_KERNEL, 2)
    remp.remp_alloc_dst_blocks(plan, [total] * 4, 0, torch.empty_like(d_bt))
    s_sh, d_sh = remp.make_shards(d_src, [pool] * 2), remp.make_shards(d_dst, [total] * 4)
    with pytest.raises(remp.RempError) as ei:                         # device 0 would read rank 1's shard from device 1
        remp.remp_migrate_kv_exchange(plan, [0, 1], [0, 0, 0, 0], 0, s_sh, d_sh)
    assert ei.value.status == remp.REMP_ERR_INVALID_ARG
    assert all(bool((t == POISON_BYTE).all()) for t in d_dst)
    remp.remp_migrate_kv_exchange(plan, [0, 0], [0, 0, 0, 0], 0, s_sh, d_sh)      # everything local: allowed
    assert remp.remp_plan_status(plan) == remp.REMP_OK
    remp.remp_plan_destroy(plan)
    for r in range(4):
        assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r])


def test_a_switch_replays_from_a_cuda_graph():
    """alloc + migrate of a switch are two kernel launches that only enqueue: captured once into a CUDA graph and
    replayed on fresh inputs, the replay gives the oracle's tables and bytes for the inputs present at replay time."""
    m = Shape(3, 4, 64, 16, 2)
    S, D = Topo(2, 1), Topo(4, 1)
    lens, bt, pool = small_workload(m, 12, 120, seed=5)
    lens2 = np.maximum(lens - 17, 0).astype(np.int32)              # other lengths, same table shape
    ns, nd = 2, 4
    rng = np.random.default_rng(3)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    cap = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [cap] * nd
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((orc.shard_bytes(D, m, r, cap),), POISON_BYTE, dtype=torch.uint8, device="cuda") for r in range(nd)]
    d_dbt = torch.full_like(d_bt, -7)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    s_sh, d_sh = remp.make_shards(d_src, [pool] * ns), remp.make_shards(d_dst, dst_nb)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                                   # first use creates the plan's scratch
        remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt, want_total=False)
        remp.remp_migrate_kv(plan, s_sh, d_sh)
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    launches0 = remp.remp_kernel_launch_count()
    with torch.cuda.graph(g, stream=side):
        remp.remp_alloc_dst_blocks(plan, dst_nb, 0, d_dbt, want_total=False)
        remp.remp_migrate_kv(plan, s_sh, d_sh)
    assert remp.remp_kernel_launch_count() - launches0 == 2
    for cur in (lens2, lens):                                       # replay on changed, then on the first inputs
        d_lens.copy_(torch.from_numpy(cur))
        for t in d_dst:
            t.fill_(POISON_BYTE)
        d_dbt.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert remp.remp_plan_status(plan) == remp.REMP_OK
        want = oracle_run(S, D, m, cur, bt, src, [pool] * ns, dst_nb)
        assert np.array_equal(d_dbt.cpu().numpy(), want[1])
        for r in range(nd):
            assert np.array_equal(d_dst[r].cpu().numpy(), want[0][r]), r
    remp.remp_plan_destroy(plan)



def _golden_rows(name):
    import os
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


@pytest.mark.parametrize("model", [r[0] for r in _golden_rows("model_shapes.txt")])
@pytest.mark.parametrize("layout", ["head", "token"])
def test_every_switch_of_the_papers_matrix_is_bit_exact(model, layout):
    """The paper's source-target matrix (section 4.2: 42 ordered pairs of seven layouts) on the layer and KV-head
    counts of its four models (section 4.1), narrow heads and short blocks so that the oracle stays fast: pools,
    tables and totals equal the oracle's on every switch, with head-major and with token-major blocks."""
    L, Hk = next((int(r[1]), int(r[2])) for r in _golden_rows("model_shapes.txt") if r[0] == model)
    layouts = [Topo(int(a), int(b)) for a, b in _golden_rows("layouts.txt")]
    m = Shape(L, Hk, 16, 4, 2)
    lens, bt, pool = small_workload(m, 6, 23, seed=17, zero_fraction=0.1)
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_dbt = torch.empty_like(d_bt)
    rng = np.random.default_rng(5)
    n = 0
    for S in layouts:
        ns = S.tp * S.pp
        src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
        d_src = [to_dev(b) for b in src]
        for D in layouts:
            if (S.tp, S.pp) == (D.tp, D.pp):
                continue
            nd = D.tp * D.pp
            dst_nb = [total + 2] * nd
            want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], m.block_size, 1, dst_nb)
            want = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
            assert orc.migrate(S, D, m, lens, bt, want_dbt, src, [pool] * ns, want, dst_nb, nthreads=4,
                               src_layout=layout, dst_layout=layout) == 0
            d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want]
            plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
            assert remp.remp_alloc_dst_blocks(plan, dst_nb, 1, d_dbt) == want_total
            remp.remp_migrate_kv(plan, remp.make_shards(d_src, [pool] * ns, [_layout_strides(S, m, layout)] * ns),
                                 remp.make_shards(d_dst, dst_nb, [_layout_strides(D, m, layout)] * nd))
            assert remp.remp_plan_status(plan) == remp.REMP_OK
            remp.remp_plan_destroy(plan)
            assert np.array_equal(d_dbt.cpu().numpy(), want_dbt), (model, str(S), str(D))
            for r in range(nd):
                assert np.array_equal(d_dst[r].cpu().numpy(), want[r]), (model, str(S), str(D), r)
            n += 1
    assert n == 42
