"""Two processes (gloo, CPU) carry out the cross-device exchange of a re-sharding the way two GPUs would:
each owns the shards of the ranks mapped to it, takes its receive and send lists from the library's
remp_plan_partition (host-only call), ships every send item's head slices with dist.send, places what it
receives, and copies its local items itself. Every rank's destination pools must equal the oracle's, bit
for bit. No GPU and no kernel is involved: this covers the partitioning logic of the multi-GPU path."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class _FakeTensor:
    """Stands in for the device tables: remp_plan_create only records the pointers."""
    def __init__(self, shape):
        self.shape, self.is_cuda, self.dtype = shape, True, "torch.int32"

    def dim(self):
        return len(self.shape)

    def is_contiguous(self):
        return True

    def data_ptr(self):
        return 0x1000


def _views(T, m, bufs, nb):
    from oracle import brute
    return [brute.shard_view(T, m, r, bufs[r], nb[r]) for r in range(T.tp * T.pp)]


def _worker(rank, world, port, q, case):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2606_18741_b200 as remp
    from oracle import brute, remp_oracle as orc
    from paper_2606_18741_b200.synth import POISON_BYTE, Shape, Topo, make_workload, small_workload
    from tests import helpers as H

    if case == "tiny":
        w = make_workload("tiny")
        m, S, D = w.shape, w.chain[0], w.chain[1]                    # TP1PP1 -> TP2PP2
        lens, bt, pool = w.seq_lens, w.block_tables, w.num_src_blocks
    else:                                                            # replication and uneven stages
        m, S, D = Shape(5, 2, 8, 4, 2), Topo(2, 2), Topo(4, 3)
        lens, bt, pool = small_workload(m, 6, 30, seed=9, zero_fraction=0.2)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    sdev = [r % world for r in range(ns)]
    ddev = [(r + 1) % world for r in range(nd)]
    G = H.random_global(m, pool, 3)
    src_all = H.shards_from_global(S, m, G)                          # the same seeded bytes in every process ...
    src = [b if sdev[r] == rank else None for r, b in enumerate(src_all)]   # ... but a rank only uses its own
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    dst_nb = [total + 1] * nd
    dbt, _off, _tot = orc.alloc(lens, bt.shape[1], m.block_size, 0, dst_nb)
    dst = [np.full(orc.shard_bytes(D, m, r, dst_nb[r]), POISON_BYTE, dtype=np.uint8) if ddev[r] == rank else None
           for r in range(nd)]

    plan = remp.remp_plan_create(S, D, m, _FakeTensor((len(lens),)), _FakeTensor(bt.shape))
    recv, send = remp.remp_plan_partition(plan, sdev, ddev, rank)
    remp.remp_plan_destroy(plan)

    src_ids = H.flat_live_ids(m, lens, bt)
    dst_ids = H.flat_live_ids(m, lens, dbt)
    sb, db = brute.stage_bounds(S, m.num_layers), brute.stage_bounds(D, m.num_layers)

    def src_slices(item):
        s_, _d, l, lo, hi, _o = (int(x) for x in item)
        v = brute.shard_view(S, m, s_, src[s_], pool)
        h0 = brute.owned_heads(S, m.num_kv_heads, s_ % S.tp)[0]
        return np.ascontiguousarray(v[l - sb[s_ // S.tp][0], :, src_ids, lo - h0:hi - h0])   # [live][2][heads][bs][De]

    def place(item, data):
        _s, d_, l, lo, hi, _o = (int(x) for x in item)
        v = brute.shard_view(D, m, d_, dst[d_], dst_nb[d_])
        h0 = brute.owned_heads(D, m.num_kv_heads, d_ % D.tp)[0]
        for kv in range(2):
            v[l - db[d_ // D.tp][0], kv, dst_ids, lo - h0:hi - h0] = data[:, kv]

    # sends first (non-blocking), then the receives in the sender's order, then the local copies
    pending = []
    for it in send:
        pending.append(dist.isend(torch.from_numpy(src_slices(it)), dst=int(it[5])))
    for peer in range(world):
        if peer == rank:
            continue
        for it in recv[recv[:, 5] == peer]:
            shape = (len(src_ids), 2, int(it[4] - it[3]), m.block_size, m.head_dim * m.elem_bytes)
            buf = torch.empty(shape, dtype=torch.uint8)
            dist.recv(buf, src=peer)
            place(it, buf.numpy())
    for it in recv[recv[:, 5] == rank]:
        place(it, src_slices(it))
    for p in pending:
        p.wait()

    want = [np.full(orc.shard_bytes(D, m, r, dst_nb[r]), POISON_BYTE, dtype=np.uint8) for r in range(nd)]
    assert orc.migrate(S, D, m, lens, bt, dbt, src_all, [pool] * ns, want, dst_nb) == 0
    ok = all(np.array_equal(dst[r], want[r]) for r in range(nd) if ddev[r] == rank)
    sent_heads = int((send[:, 4] - send[:, 3]).sum())
    got_heads = int((recv[recv[:, 5] != rank][:, 4] - recv[recv[:, 5] != rank][:, 3]).sum())
    q.put((rank, ok, sent_heads, got_heads, len(recv), len(send)))
    dist.barrier()
    dist.destroy_process_group()


def _run(case):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000 + (0 if case == "tiny" else 1)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q, case)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(r[1] for r in res), res                       # both ranks match the oracle bit for bit
    assert res[0][2] == res[1][3] and res[1][2] == res[0][3]  # what one sends the other receives
    assert res[0][2] + res[1][2] > 0                         # something did cross
    return res


def test_two_ranks_exchange_the_tiny_configuration():
    _run("tiny")


def test_two_ranks_exchange_with_replication_and_uneven_stages():
    _run("replicated")
