"""The cross-GPU exchange carried out by TWO PROCESSES: each owns half of the logical ranks, publishes its source
pools as CUDA IPC handles, and pulls what its destination ranks receive with remp_migrate_kv_exchange - remote
sources are read in place through the mapped handle. On this one-GPU test both processes use the same device (the
mapping, the partitioning and the kernel path are those of a two-GPU run; only the wire is missing). The
processes never wait for each other on the device: a host barrier before and after each leg is all there is.
Every process checks its own destination pools against the oracle, bit for bit."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _worker(rank, world, port, q, case):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    import paper_2606_18741_b200 as remp
    from oracle import remp_oracle as orc
    from paper_2606_18741_b200.synth import POISON_BYTE, Shape, Topo, Workload, fill_payload_numpy, make_workload, small_workload
    from tests.device_workload import ExchangeWorkload
    try:
        if case == "tiny":
            w = make_workload("tiny")
        else:                                            # 2x replication on the way, uneven stages, three legs
            m = Shape(5, 4, 64, 16, 2)
            lens, bt, pool = small_workload(m, 12, 150, seed=6, zero_fraction=0.1)
            w = Workload("case", m, [Topo(2, 2), Topo(8, 1), Topo(4, 3), Topo(1, 1)], lens, bt, pool, 5)
        xw = ExchangeWorkload(w, rank, world)
        # the oracle's own chain, whole cache, from the same seeded payload
        m = w.shape
        cur = []
        for r in range(w.chain[0].tp * w.chain[0].pp):
            b = np.empty(orc.shard_bytes(w.chain[0], m, r, w.num_src_blocks), dtype=np.uint8)
            fill_payload_numpy(b, xw.seed, r)
            cur.append(b)
        cur_bt, cur_nb = w.block_tables, [w.num_src_blocks] * len(cur)
        ok = True
        for leg in range(len(w.chain) - 1):
            S, D = w.chain[leg], w.chain[leg + 1]
            nd = D.tp * D.pp
            dst_nb = [w.live_blocks] * nd
            dbt, _off, _tot = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, dst_nb)
            nxt = [np.full(orc.shard_bytes(D, m, r, dst_nb[r]), POISON_BYTE, dtype=np.uint8) for r in range(nd)]
            assert orc.migrate(S, D, m, w.seq_lens, cur_bt, dbt, cur, cur_nb, nxt, dst_nb) == 0
            plan, _ms = xw.run_leg(leg)
            ok = ok and remp.remp_plan_status(plan) == remp.REMP_OK
            remp.remp_plan_destroy(plan)
            ok = ok and np.array_equal(xw.d_bt[leg + 1].cpu().numpy(), dbt)
            for r, t in xw.pools[leg + 1].items():
                ok = ok and np.array_equal(t.cpu().numpy(), nxt[r])
            cur, cur_bt, cur_nb = nxt, dbt, dst_nb
        held = sum(len(p) for p in xw.pools)
        xw.close()
        q.put((rank, bool(ok), held, ""))
    except Exception as exc:                              # reported to the parent, which fails the test
        q.put((rank, False, 0, repr(exc)))
    dist.barrier()
    dist.destroy_process_group()
    # everything is unmapped and collected (ExchangeWorkload.close): leave without running the interpreter's
    # teardown, whose order of destroying CUDA IPC bookkeeping is not ours to control
    q.close()
    q.join_thread()
    sys.stdout.flush()
    os._exit(0)


@pytest.mark.parametrize("case", ["tiny", "chain"])
def test_two_processes_exchange_through_ipc_mapped_pools(case):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000 + (0 if case == "tiny" else 1)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q, case)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert all(r[1] for r in res), res
    assert res[0][2] > 0 and res[1][2] > 0                 # both processes held shards
