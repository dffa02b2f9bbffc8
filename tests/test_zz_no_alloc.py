"""remp_remap_tables_noalloc against the oracle's allocator and remp_alloc_dst_blocks (collected last on purpose).

The no-allocation entry point serves callers that cannot call cudaMalloc when a topology switch happens
(all HBM already handed to KV pools, a latency-critical loop, a fixed memory budget); its scratch is a
fixed array inside the library that every call shares and that keeps the previous call's contents. So the
check runs two different inputs back to back - the second smaller, so stale offsets of the first are still
in the array - and each must give exactly the tables and total the oracle's serial allocator gives, which is
also what the allocating entry point gives. A last test watches the device's free memory around a call: the
entry point exists because its callers cannot allocate, so it must not allocate either.
"""
import numpy as np
import pytest
import torch

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import Shape, Topo

pytestmark = pytest.mark.gpu


def _inputs(n, max_len, block_size, seed):
    rng = np.random.default_rng(seed)
    lens = rng.integers(0, max_len + 1, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // block_size)
    maxb = int(need.max()) + 3
    total = int(need.sum())
    bt = np.full((n, maxb), -1, dtype=np.int32)
    ids = rng.permutation(total + 5)[:total].astype(np.int32)
    pos = 0
    for s in range(n):
        bt[s, :need[s]] = ids[pos:pos + need[s]]
        pos += need[s]
    return lens, bt, total


def _reference(lens, bt, block_size, base, cap):
    """The existing entry point: plan + remp_alloc_dst_blocks."""
    m = Shape(1, 1, 16, block_size, 1)
    d_lens, d_bt = torch.from_numpy(lens).cuda(), torch.from_numpy(bt).cuda()
    out = torch.full_like(d_bt, -9)
    plan = remp.remp_plan_create(Topo(1, 1), Topo(1, 1), m, d_lens, d_bt)
    try:
        total = remp.remp_alloc_dst_blocks(plan, [cap], base, out)
    finally:
        remp.remp_plan_destroy(plan)
    return out.cpu().numpy(), total


def _noalloc(lens, bt, block_size, base, cap):
    d_lens = torch.from_numpy(lens).cuda()
    out = torch.full(bt.shape, -9, dtype=torch.int32, device="cuda")
    result = torch.full((2,), -9, dtype=torch.int32, device="cuda")
    remp.remp_remap_tables_noalloc(d_lens, bt.shape[1], block_size, base, cap, out, result)
    torch.cuda.synchronize()
    total, status = result.cpu().tolist()
    return out.cpu().numpy(), total, status


def test_noalloc_matches_alloc_dst_blocks_twice_in_a_row():
    first = _inputs(3000, 700, 16, seed=1)          # spans three scan tiles
    second = _inputs(517, 90, 16, seed=2)           # smaller: the array still holds the first call's offsets
    for (lens, bt, total), base in ((first, 5), (second, 0)):
        orc_bt, _off, orc_total = orc.alloc(lens, bt.shape[1], 16, base, [base + total])
        got_bt, got_total, status = _noalloc(lens, bt, 16, base, base + total)
        assert status == 0
        assert got_total == orc_total == total
        assert np.array_equal(got_bt, orc_bt)        # integer output: exact, against the oracle
        want_bt, want_total = _reference(lens, bt, 16, base, base + total)
        assert want_total == got_total and np.array_equal(got_bt, want_bt)   # and against the allocating entry point


def test_noalloc_reports_capacity_and_rejects_oversize():
    lens, bt, total = _inputs(100, 50, 16, seed=3)
    got_bt, got_total, status = _noalloc(lens, bt, 16, 0, total - 1)
    assert status & 1 and (got_bt == -9).all()       # capacity exceeded: tables untouched
    # a clean call afterwards is not affected by the failed one
    want_bt, want_total = _reference(lens, bt, 16, 0, total)
    got_bt, got_total, status = _noalloc(lens, bt, 16, 0, total)
    assert status == 0 and got_total == want_total and np.array_equal(got_bt, want_bt)
    n = remp.REMP_NOALLOC_MAX_SEQS + 1
    d_lens = torch.zeros(n, dtype=torch.int32, device="cuda")
    out = torch.zeros((n, 1), dtype=torch.int32, device="cuda")
    result = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(remp.RempError) as ei:
        remp.remp_remap_tables_noalloc(d_lens, 1, 16, 0, 10, out, result)
    assert ei.value.status == remp.REMP_ERR_INVALID_ARG and "REMP_NOALLOC_MAX_SEQS" in str(ei.value)


def test_noalloc_takes_no_device_memory():
    """Free device memory, as the driver reports it, is the same before and after a call (after one warm-up call
    that loads the kernels): neither the runtime nor a memory pool grew."""
    lens, bt, total = _inputs(2000, 300, 16, seed=4)
    d_lens = torch.from_numpy(lens).cuda()
    out = torch.empty(bt.shape, dtype=torch.int32, device="cuda")
    result = torch.empty(2, dtype=torch.int32, device="cuda")
    remp.remp_remap_tables_noalloc(d_lens, bt.shape[1], 16, 0, total, out, result)
    torch.cuda.synchronize()
    free0, _t = torch.cuda.mem_get_info()
    launches0 = remp.remp_kernel_launch_count()
    for _ in range(3):
        remp.remp_remap_tables_noalloc(d_lens, bt.shape[1], 16, 0, total, out, result)
    torch.cuda.synchronize()
    free1, _t = torch.cuda.mem_get_info()
    assert free1 == free0
    assert remp.remp_kernel_launch_count() - launches0 == 6          # two kernels per call
    orc_bt, _off, orc_total = orc.alloc(lens, bt.shape[1], 16, 0, [total])
    assert result.cpu().tolist() == [orc_total, 0] and np.array_equal(out.cpu().numpy(), orc_bt)
