"""world_size-2 run of the benchmark's multi-rank logic on CPU (gloo): replicas only, no data-path
collective; the job value is all ranks' bytes over the slowest rank's time."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2606_18741_b200.synth import make_workload
    # every rank builds its own replica (seed = rank) and would time it on its own GPU
    w = make_workload("tiny", seed=rank)
    local_bytes = 1000 + 10 * w.live_blocks
    ms, total = bench.reduce_job(5.0 + rank, local_bytes, None)
    all_bytes = [None] * world
    dist.all_gather_object(all_bytes, local_bytes)
    q.put((rank, ms, total, sum(all_bytes), w.live_blocks))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replicas_reduce_max_time_and_sum_bytes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, tot0, want0, live0), (r1, ms1, tot1, want1, live1) = res
    assert ms0 == ms1 == 6.0                       # the slowest rank sets the time
    assert tot0 == tot1 == want0 == want1          # bytes of all replicas
    assert live0 != live1                          # the replicas are different workloads


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_job(3.5, 77, None) == (3.5, 77)
