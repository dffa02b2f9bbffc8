"""Randomised GPU parity: random model shapes, topology pairs (incl. replication, explicit uneven stages),
block layouts on either side, allocation flavours, kernel options and - every other case - the destination ranks
spread over 1..4 logical devices (remp_migrate_kv_exchange, one call per device) - always bit-exact against the
oracle."""
import os

import numpy as np
import pytest
import torch

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import POISON_BYTE, Shape, Topo
from tests import helpers as H
from tests.gpu_harness import to_dev

pytestmark = pytest.mark.gpu


def _random_topo(rng, L, Hh):
    tps = [t for t in (1, 2, 3, 4, 6, 8, 12, 16, 24) if (Hh % t == 0 if t <= Hh else t % Hh == 0)]
    tp = int(rng.choice(tps))
    pp = int(rng.integers(1, min(L, 5) + 1))
    if pp > 1 and rng.random() < 0.4:                      # explicit uneven stages
        cuts = sorted(rng.choice(np.arange(1, L), size=pp - 1, replace=False).tolist())
        return Topo(tp, pp, tuple([0] + cuts + [L]))
    return Topo(tp, pp)


def _random_tables(rng, n, bs, pool_factor, max_len, share):
    lens = rng.integers(0, max_len + 1, size=n).astype(np.int32)
    need = -(-lens.astype(np.int64) // bs)
    total = int(need.sum())
    pool = max(1, int(total * pool_factor) + 1)
    maxb = int(need.max(initial=1)) + int(rng.integers(0, 3))
    bt = np.full((n, max(1, maxb)), -1, dtype=np.int32)
    free = list(rng.permutation(pool))
    for s in range(n):
        k = 0
        if share and s and rng.random() < 0.5:
            o = int(rng.integers(0, s))
            k = int(rng.integers(0, min(need[s], need[o]) + 1))
            bt[s, :k] = bt[o, :k]
        for j in range(k, need[s]):
            bt[s, j] = free.pop()
    return lens, bt, pool


OPTION_SETS = [{}, {remp.REMP_OPT_SCHEDULE: 1}, {remp.REMP_OPT_KERNEL: 2}, {remp.REMP_OPT_VEC_BYTES: 32},
               {remp.REMP_OPT_CHUNK_BYTES: 2048, remp.REMP_OPT_TILE_ITEMS: 3}, {remp.REMP_OPT_CTAS_PER_SM: 1},
               {remp.REMP_OPT_ORDER: 1}]


@pytest.mark.parametrize("seed", range(int(os.environ.get("REMP_RANDOM_CASES", "40"))))
def test_random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    L = int(rng.integers(1, 9))
    Hh = int(rng.choice([1, 2, 4, 6, 8, 12]))
    D_ = int(rng.choice([16, 32, 40, 64, 128]))
    e = int(rng.choice([1, 2, 4]))
    bs = int(rng.choice([4, 8, 16, 32]))
    if (bs * D_ * e) % 16:
        bs = 16
    m = Shape(L, Hh, D_, bs, e)
    S, D = _random_topo(rng, L, Hh), _random_topo(rng, L, Hh)
    flavour = ["plain", "preempt", "shared"][seed % 3]
    lens, bt, pool = _random_tables(rng, int(rng.integers(1, 40)), bs, 1.3, 6 * bs, share=(flavour == "shared"))
    src_layout = str(rng.choice(["head", "token"]))
    dst_layout = str(rng.choice(["head", "token"]))
    if (D_ * e) % 16:                                     # strided rows must be whole 16-byte vectors
        src_layout = dst_layout = "head"
    opts = OPTION_SETS[seed % len(OPTION_SETS)]
    ns, nd = S.tp * S.pp, D.tp * D.pp
    base = int(rng.integers(0, 4))
    need = -(-lens.astype(np.int64) // bs)
    src = [rng.integers(0, 256, size=orc.shard_bytes(S, m, r, pool), dtype=np.uint8) for r in range(ns)]
    # ---- oracle ----
    if flavour == "preempt":
        dst_nb = [base + int(0.6 * need.sum()) + (r % 2) for r in range(nd)]
        want_dbt, want_pre, want_total = orc.alloc_preempt(lens, bt.shape[1], bs, base, dst_nb)
        olens = np.where(want_pre == 0, lens, 0).astype(np.int32)
    elif flavour == "shared":
        want_dbt, want_total, _bad = orc.alloc_shared(lens, bt, bs, base, pool, [10**7] * nd)
        dst_nb = [base + want_total + (r % 2) for r in range(nd)]
        olens = lens
    else:
        dst_nb = [base + int(need.sum()) + (r % 3) for r in range(nd)]
        want_dbt, _off, want_total = orc.alloc(lens, bt.shape[1], bs, base, dst_nb)
        olens = lens
    want = H.poison_like([orc.shard_bytes(D, m, r, dst_nb[r]) for r in range(nd)])
    assert orc.migrate(S, D, m, olens, bt, want_dbt, src, [pool] * ns, want, dst_nb, nthreads=2,
                       src_layout=src_layout, dst_layout=dst_layout) == 0
    # ---- CUDA path ----
    de = D_ * e

    def strides(T, lay):
        hl = orc.heads_per_rank(T, Hh)
        return {"head": de, "token": hl * de} if lay == "token" else {}

    d_lens, d_bt = to_dev(lens), to_dev(bt)
    d_src = [to_dev(b) for b in src]
    d_dst = [torch.full((len(b),), POISON_BYTE, dtype=torch.uint8, device="cuda") for b in want]
    d_dbt = torch.full_like(d_bt, -7)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    try:
        for k_, v_ in opts.items():
            remp.remp_plan_set_option(plan, k_, v_)
        if flavour == "preempt":
            d_pre = torch.empty(len(lens), dtype=torch.int32, device="cuda")
            total, npre = remp.remp_alloc_dst_blocks_preempt(plan, dst_nb, base, d_dbt, d_pre)
            assert np.array_equal(d_pre.cpu().numpy(), want_pre) and npre == int(want_pre.sum())
        elif flavour == "shared":
            total = remp.remp_alloc_dst_blocks_shared(plan, dst_nb, base, pool, d_dbt)
        else:
            total = remp.remp_alloc_dst_blocks(plan, dst_nb, base, d_dbt)
        s_sh = remp.make_shards(d_src, [pool] * ns, [strides(S, src_layout)] * ns)
        d_sh = remp.make_shards(d_dst, dst_nb, [strides(D, dst_layout)] * nd)
        if seed % 2 == 1 and opts.get(remp.REMP_OPT_KERNEL) != 2:
            ndev = int(rng.integers(1, 5))                 # random rank -> device maps; every device in turn
            sdev = [int(x) for x in rng.integers(0, ndev, size=ns)]
            ddev = [int(x) for x in rng.integers(0, ndev, size=nd)]
            for q in range(ndev):
                remp.remp_migrate_kv_exchange(plan, sdev, ddev, q, s_sh, d_sh)
        else:
            remp.remp_migrate_kv(plan, s_sh, d_sh)
        assert remp.remp_plan_status(plan) == remp.REMP_OK, remp.remp_last_error()
    finally:
        remp.remp_plan_destroy(plan)
    tag = (str(S), S.layer_start, str(D), D.layer_start, m, flavour, src_layout, dst_layout, opts)
    assert total == want_total, tag
    assert np.array_equal(d_dbt.cpu().numpy(), want_dbt), tag
    for r in range(nd):
        assert np.array_equal(d_dst[r].cpu().numpy(), want[r]), (tag, r)
