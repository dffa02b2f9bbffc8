"""GPU parity at the benchmark's sizes, in the launch configuration bench.py times (default options).

Whole pools do not fit the oracle's time budget, so each transition is checked by
  (a) block tables, ids and total against the oracle's serial allocator (exact);
  (b) sampled head slices: the oracle's ownership and offset functions locate, one by one, where in the
      ORIGINAL source pools a destination slice must come from, and the seeded payload generator gives the
      expected bytes (also through chained transitions, since ids stay logical-block ordered);
  (c) whole layers re-sharded by the oracle alone, transition after transition, starting from that layer's
      source slabs regenerated on the host from the seeded payload (nothing the GPU produced is fed to it);
  (d) properties that hold at any size: wrap-around word sums of live source and destination blocks
      agree (times the replication), slack destination blocks keep the poison fill, replicas are equal,
      and the source pools are unchanged.
"""
import gc
import os

import numpy as np
import pytest
import torch

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from tests.device_workload import DeviceWorkload
from paper_2606_18741_b200.synth import POISON_BYTE, fill_payload_torch, make_workload, payload_bytes
from tests import helpers as H

pytestmark = pytest.mark.gpu

SLACK = 3
TEST_BUDGET_GIB = float(os.environ.get("REMP_TEST_BUDGET_GIB", "24"))


def _sum_words(t: torch.Tensor) -> int:
    return int(t.view(torch.int64).sum().item())


def _plane_view(T, m, r, pool: torch.Tensor, nb: int) -> torch.Tensor:
    """[local layer][2][block][bytes of all local heads] view of a device pool."""
    hl = orc.heads_per_rank(T, m.num_kv_heads)
    blk = hl * m.block_size * m.head_dim * m.elem_bytes
    return pool.view(-1, 2, nb, blk)



def _host_source_slab(dw, rank, layer_local, lb):
    """Layer slab of a source pool regenerated on the host from the seeded payload (no device involved)."""
    from paper_2606_18741_b200.synth import payload_bytes as pb
    return pb(dw.seed, rank, layer_local * lb, lb)


def _oracle_chain_layer(dw, l, upto_leg, layouts=None):
    """Layer l through the oracle alone: legs 0..upto_leg starting from the host-generated source payload.
    Returns (slabs per destination TP rank of the last leg, tables after the last leg)."""
    w, m = dw.w, dw.m
    L = m.num_layers
    lay = layouts or ["head"] * len(w.chain)
    S = w.chain[0]
    ps = orc.pp_owner(S, L, l)
    cur = []
    for t in range(S.tp):
        r = orc.rank_of(S, ps, t)
        lb = orc.layer_slab_bytes(S, m, dw.nb[0][r])
        cur.append(_host_source_slab(dw, r, l - orc.stage_first(S, L, ps), lb))
    cur_bt = w.block_tables
    for leg in range(upto_leg + 1):
        S, D = w.chain[leg], w.chain[leg + 1]
        ps, pd = orc.pp_owner(S, L, l), orc.pp_owner(D, L, l)
        nbS = [dw.nb[leg][orc.rank_of(S, ps, t)] for t in range(S.tp)]
        nbD = [dw.nb[leg + 1][orc.rank_of(D, pd, t)] for t in range(D.tp)]
        dbt, _off, _tot = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, dw.nb[leg + 1])
        nxt = [np.full(orc.layer_slab_bytes(D, m, nbD[t]), POISON_BYTE, dtype=np.uint8) for t in range(D.tp)]
        assert orc.migrate_layer(S, D, m, w.seq_lens, cur_bt, dbt, cur, nbS, nxt, nbD, src_layout=lay[leg],
                                 dst_layout=lay[leg + 1]) == 0
        cur, cur_bt = nxt, dbt
    return cur, cur_bt


def _check_every_layer(dw: DeviceWorkload):
    """Every layer of every leg through the oracle, one layer at a time (host memory stays at a few slabs).
    The oracle runs its own chain: leg 0 from the layer's source slabs (read back from the source pools, whose
    payload the sampled slices and the host-generated layers of _check_leg tie to the seeded generator), every
    later leg from the oracle's own previous result; each result is compared with the device pool byte for byte."""
    w, m = dw.w, dw.m
    L = m.num_layers
    tables = [w.block_tables]
    for leg in range(dw.num_legs):
        dbt, _off, _tot = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, dw.nb[leg + 1])
        tables.append(dbt)
    for l in range(L):
        S = w.chain[0]
        ps = orc.pp_owner(S, L, l)
        cur = []
        for t in range(S.tp):
            r = orc.rank_of(S, ps, t)
            lb = orc.layer_slab_bytes(S, m, dw.nb[0][r])
            o = (l - orc.stage_first(S, L, ps)) * lb
            cur.append(dw.pools[0][r][o:o + lb].cpu().numpy())
        for leg in range(dw.num_legs):
            S, D = w.chain[leg], w.chain[leg + 1]
            ps, pd = orc.pp_owner(S, L, l), orc.pp_owner(D, L, l)
            nbS = [dw.nb[leg][orc.rank_of(S, ps, t)] for t in range(S.tp)]
            nbD = [dw.nb[leg + 1][orc.rank_of(D, pd, t)] for t in range(D.tp)]
            nxt = [np.full(orc.layer_slab_bytes(D, m, nbD[t]), POISON_BYTE, dtype=np.uint8) for t in range(D.tp)]
            assert orc.migrate_layer(S, D, m, w.seq_lens, tables[leg], tables[leg + 1], cur, nbS, nxt, nbD) == 0
            for t in range(D.tp):
                r = orc.rank_of(D, pd, t)
                lb = orc.layer_slab_bytes(D, m, nbD[t])
                o = (l - orc.stage_first(D, L, pd)) * lb
                assert np.array_equal(dw.pools[leg + 1][r][o:o + lb].cpu().numpy(), nxt[t]), (leg, l, t)
            cur = nxt


def _check_leg(dw: DeviceWorkload, leg: int, flatA: np.ndarray, rng, n_samples: int, layers):
    w, m = dw.w, dw.m
    A, S, D = w.chain[0], w.chain[leg], w.chain[leg + 1]
    L, Hh = m.num_layers, m.num_kv_heads
    hs = m.block_size * m.head_dim * m.elem_bytes
    live = dw.live
    nbD, nbS, nbA = dw.nb[leg + 1], dw.nb[leg], dw.nb[0]

    # (a) tables
    want_dbt, _off, want_total = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, nbD)
    assert want_total == live
    assert np.array_equal(dw.d_bt[leg + 1].cpu().numpy(), want_dbt)

    # (b) sampled slices, traced back to the original pools
    offs, exp = [], []
    for _ in range(n_samples):
        r = int(rng.integers(0, D.tp * D.pp))
        p, t = divmod(r, D.tp)
        l = int(rng.integers(orc.stage_first(D, L, p), orc.stage_first(D, L, p + 1)))
        kv = int(rng.integers(0, 2))
        k = int(rng.integers(0, live))
        lo, hi = orc.head_range(D, Hh, t)
        h = int(rng.integers(lo, hi))
        d_off = orc.offset(D, m, r, nbD[r], l, kv, k, h)
        ra = orc.rank_of(A, orc.pp_owner(A, L, l), orc.tp_owner(A, Hh, h))
        a_off = orc.offset(A, m, ra, nbA[ra], l, kv, int(flatA[k]), h)
        assert d_off >= 0 and a_off >= 0
        offs.append((r, d_off))
        exp.append(payload_bytes(dw.seed, ra, a_off, hs))
    got = torch.stack([dw.pools[leg + 1][r][o:o + hs] for r, o in offs]).cpu().numpy()
    assert np.array_equal(got, np.stack(exp))

    # (c) whole layers through the oracle alone (its own chain from the host-generated source payload)
    src_bt = dw.d_bt[leg].cpu().numpy()
    for l in layers:
        pd = orc.pp_owner(D, L, l)
        want, chain_bt = _oracle_chain_layer(dw, l, leg)
        assert np.array_equal(chain_bt, want_dbt)
        for t in range(D.tp):
            r = orc.rank_of(D, pd, t)
            lb = orc.layer_slab_bytes(D, m, nbD[r])
            o = (l - orc.stage_first(D, L, pd)) * lb
            assert np.array_equal(dw.pools[leg + 1][r][o:o + lb].cpu().numpy(), want[t]), (leg, l, t)

    # (d) properties
    src_ids = torch.from_numpy(H.flat_live_ids(m, w.seq_lens, src_bt)).cuda()
    repS, repD = orc.rep(S, Hh), orc.rep(D, Hh)
    src_sum = 0
    for r in range(S.tp * S.pp):
        if (r % S.tp) % repS:
            continue                                            # only the lowest replica is the source
        v = _plane_view(S, m, r, dw.pools[leg][r], nbS[r])
        for l0 in range(v.shape[0]):                            # layer by layer bounds the temporary
            src_sum += _sum_words(v[l0].index_select(1, src_ids).contiguous())
    dst_sum = 0
    for r in range(D.tp * D.pp):
        v = _plane_view(D, m, r, dw.pools[leg + 1][r], nbD[r])
        dst_sum += _sum_words(v[:, :, :live].contiguous())
        assert bool((v[:, :, live:] == POISON_BYTE).all()), "a slack destination block was written"
    mask = (1 << 64) - 1
    assert (dst_sum & mask) == ((src_sum * repD) & mask)
    if repD > 1:
        for r in range(D.tp * D.pp):
            r0 = r - (r % D.tp) % repD
            if r != r0:
                assert torch.equal(dw.pools[leg + 1][r], dw.pools[leg + 1][r0])


def _run_config(name, budget_bytes=None, n_samples=1500, every_layer=False):
    w = make_workload(name, seed=0, budget_bytes=budget_bytes)
    need = 0
    dw = DeviceWorkload(w, dst_slack_blocks=SLACK)
    try:
        free, _tot = torch.cuda.mem_get_info()
        rng = np.random.default_rng(42)
        flatA = H.flat_live_ids(w.shape, w.seq_lens, w.block_tables)
        src_sums = [_sum_words(t) for t in dw.pools[0]]
        plans = [dw.run_leg(i) for i in range(dw.num_legs)]
        torch.cuda.synchronize()
        for p in plans:
            assert remp.remp_plan_status(p) == remp.REMP_OK, remp.remp_last_error()
            remp.remp_plan_destroy(p)
        L = w.shape.num_layers
        for leg in range(dw.num_legs):
            S, D = w.chain[leg], w.chain[leg + 1]
            edges = {0, L - 1}
            for T in (S, D):                       # layers on both sides of a stage boundary
                for p in range(1, T.pp):
                    b = orc.stage_first(T, L, p)
                    edges.update((b - 1, b))
            layers = sorted(edges)[:4]
            _check_leg(dw, leg, flatA, rng, n_samples, layers)
        if every_layer:
            _check_every_layer(dw)
        assert [_sum_words(t) for t in dw.pools[0]] == src_sums           # source untouched
    finally:
        del dw
        gc.collect()
        torch.cuda.empty_cache()
    return w


def test_70b_gqa_full_size():
    """80 layers, 8 KV heads, ~97k tokens, 31.8 GB live: TP4PP2 -> TP8PP1 -> TP2PP4 (4 KiB runs). Every layer of
    both legs goes through the oracle."""
    w = _run_config("70b_gqa", every_layer=True)
    assert w.live_blocks > 5000 and int(w.seq_lens.max()) <= 32768


def test_fp8_stress_full_size():
    """2048 short sequences, block_size 32, 1-byte elements: TP2PP1 -> TP16PP1 (2x replication) -> TP1PP8. Every
    layer of both legs goes through the oracle."""
    w = _run_config("fp8_stress", every_layer=True)
    assert w.num_seqs == 2048 and int(w.seq_lens.max()) <= 63


def test_7b_mha_churned_tables():
    """32 layers, 32 KV heads, fragmented tables: TP1PP1 -> TP2PP1 -> TP4PP1 (64 and 32 KiB runs)."""
    w = _run_config("7b_mha", budget_bytes=int(TEST_BUDGET_GIB * (1 << 30)))
    assert w.notes["adjacent_fraction"] < 0.9


def test_8b_gqa_regroup():
    """32 layers, 8 KV heads: TP2PP2 -> TP4PP1 -> TP1PP4 -> TP1PP2 (the last leg moves whole blocks)."""
    _run_config("8b_gqa", budget_bytes=int(TEST_BUDGET_GIB * (1 << 30)))


def test_layerwise_streaming_fits_a_cache_that_two_copies_would_not():
    """Section 3.4.4: with one allocation per (rank, layer) and the source layer released as soon as it has
    been migrated, the peak footprint is one cache plus one layer. The 8B GQA shape (512 sequences, the
    configuration whose written size does not fit next to a destination) with a cache sized so that source
    pool + destination exceed the device memory still migrates; sampled slices and whole layers are checked
    as in the other full-size tests."""
    from tests.device_workload import layer_windows, stream_leg_layerwise
    free, total_mem = torch.cuda.mem_get_info()
    # live cache L such that 1.25 L (source pool) + L (destination) > device memory > 1.25 L + a few layers
    live_target = int(0.60 * total_mem / 1.25)
    w = make_workload("8b_gqa", seed=0, budget_bytes=live_target)
    m, S, D = w.shape, w.chain[0], w.chain[1]
    L, Hh = m.num_layers, m.num_kv_heads
    hs = m.block_size * m.head_dim * m.elem_bytes
    live = w.live_blocks
    src_bytes = sum(remp.remp_shard_bytes(S, m, r, w.num_src_blocks) for r in range(S.tp * S.pp))
    dst_bytes = sum(remp.remp_shard_bytes(D, m, r, live) for r in range(D.tp * D.pp))
    assert src_bytes + dst_bytes > total_mem, "the case must not fit as two whole caches"
    wins = layer_windows(w, 1)
    keep = (0, len(wins) // 2, len(wins) - 1)
    out = stream_leg_layerwise(w, window=1, keep_windows=keep)
    try:
        layer_bytes = sum(out["src_layer_bytes"][:S.tp]) + sum(out["dst_layer_bytes"])
        assert out["peak_bytes"] <= max(src_bytes, dst_bytes) + 3 * layer_bytes + (64 << 20)
        want_dbt, _off, want_total = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, [live] * (D.tp * D.pp))
        assert want_total == live and np.array_equal(out["dst_bt"].cpu().numpy(), want_dbt)
        flatA = H.flat_live_ids(m, w.seq_lens, w.block_tables)
        rng = np.random.default_rng(7)
        # sampled destination slices traced back to the payload of the source pools
        for _ in range(600):
            r = int(rng.integers(0, D.tp * D.pp))
            p, t = divmod(r, D.tp)
            l = int(rng.integers(orc.stage_first(D, L, p), orc.stage_first(D, L, p + 1)))
            kv, k = int(rng.integers(0, 2)), int(rng.integers(0, live))
            lo, hi = orc.head_range(D, Hh, t)
            h = int(rng.integers(lo, hi))
            wi = next(i for i, (a, b) in enumerate(wins) if a <= l < b)
            d_off = orc.offset(D, m, r, live, l, kv, k, h) - (wins[wi][0] - orc.stage_first(D, L, p)) * out["dst_layer_bytes"][r]
            ra = orc.rank_of(S, orc.pp_owner(S, L, l), orc.tp_owner(S, Hh, h))
            a_off = orc.offset(S, m, ra, w.num_src_blocks, l, kv, int(flatA[k]), h)
            got = out["dst"][(r, wi)][d_off:d_off + hs].cpu().numpy()
            assert np.array_equal(got, payload_bytes(w.seed, ra, a_off, hs))
        # whole kept layers through the oracle
        for wi in keep:
            l = wins[wi][0]
            ps, pd = orc.pp_owner(S, L, l), orc.pp_owner(D, L, l)
            sslabs = [out["kept_src"][(orc.rank_of(S, ps, t), wi)].cpu().numpy() for t in range(S.tp)]
            want = [np.full(out["dst_layer_bytes"][orc.rank_of(D, pd, t)], POISON_BYTE, dtype=np.uint8) for t in range(D.tp)]
            assert orc.migrate_layer(S, D, m, w.seq_lens, w.block_tables, want_dbt, sslabs, [w.num_src_blocks] * S.tp,
                                     want, [live] * D.tp) == 0
            for t in range(D.tp):
                assert np.array_equal(out["dst"][(orc.rank_of(D, pd, t), wi)].cpu().numpy(), want[t])
    finally:
        del out
        gc.collect()
        torch.cuda.empty_cache()


def test_70b_gqa_full_size_token_major_blocks():
    """The benchmark workload with blocks kept as [token][head][dim] in every pool (256-byte rows): whole
    layers of both transitions through the oracle, tables, and the size-independent word-sum property."""
    w = make_workload("70b_gqa", seed=0)
    m = w.shape
    L = m.num_layers
    dw = DeviceWorkload(w, dst_slack_blocks=SLACK, layouts=["token"] * len(w.chain))
    try:
        plans = [dw.run_leg(i) for i in range(dw.num_legs)]
        torch.cuda.synchronize()
        for p in plans:
            assert remp.remp_plan_status(p) == remp.REMP_OK, remp.remp_last_error()
            remp.remp_plan_destroy(p)
        for leg in range(dw.num_legs):
            S, D = w.chain[leg], w.chain[leg + 1]
            nbS, nbD = dw.nb[leg], dw.nb[leg + 1]
            want_dbt, _off, want_total = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, nbD)
            assert np.array_equal(dw.d_bt[leg + 1].cpu().numpy(), want_dbt)
            src_bt = dw.d_bt[leg].cpu().numpy()
            for l in (0, L // 2 - 1, L // 2, L - 1):
                pd = orc.pp_owner(D, L, l)
                want, chain_bt = _oracle_chain_layer(dw, l, leg, layouts=["token"] * len(w.chain))
                assert np.array_equal(chain_bt, want_dbt)
                for t in range(D.tp):
                    r = orc.rank_of(D, pd, t)
                    lb = orc.layer_slab_bytes(D, m, nbD[r])
                    o = (l - orc.stage_first(D, L, pd)) * lb
                    assert np.array_equal(dw.pools[leg + 1][r][o:o + lb].cpu().numpy(), want[t]), (leg, l, t)
            # every live byte arrived: word sums over live blocks agree (layout only permutes words inside a block)
            src_ids = torch.from_numpy(H.flat_live_ids(m, w.seq_lens, src_bt)).cuda()
            src_sum = sum(_sum_words(_plane_view(S, m, r, dw.pools[leg][r], nbS[r])[l0].index_select(1, src_ids).contiguous())
                          for r in range(S.tp * S.pp) for l0 in range(L // S.pp))
            dst_sum = 0
            for r in range(D.tp * D.pp):
                v = _plane_view(D, m, r, dw.pools[leg + 1][r], nbD[r])
                dst_sum += _sum_words(v[:, :, :dw.live].contiguous())
                assert bool((v[:, :, dw.live:] == POISON_BYTE).all())
            assert (dst_sum - src_sum) % (1 << 64) == 0
    finally:
        del dw
        gc.collect()
        torch.cuda.empty_cache()


def test_70b_shape_host_resident_every_layer_through_the_oracle():
    """remp_reshard_host on a 70B-shaped cache of ~8 GB that lives in page-locked host memory (the direct path:
    the kernel reads and writes host memory): every one of the 80 layers of the result equals the oracle's, which
    reads the same host source slabs. The source is untouched, the link carried only live blocks."""
    w = make_workload("70b_gqa", seed=3, budget_bytes=8 << 30)
    m, S, D = w.shape, w.chain[0], w.chain[1]
    L = m.num_layers
    ns, nd = S.tp * S.pp, D.tp * D.pp
    src_nb, dst_nb = [w.num_src_blocks] * ns, [w.live_blocks + SLACK] * nd
    h_src = []
    for r in range(ns):
        t = torch.empty(remp.remp_shard_bytes(S, m, r, src_nb[r]), dtype=torch.uint8, pin_memory=True)
        d = torch.empty_like(t, device="cuda")
        fill_payload_torch(d, w.seed, r)                       # generated on the device (fast), brought to the host
        t.copy_(d)
        h_src.append(t)
        del d
    h_dst = [torch.full((remp.remp_shard_bytes(D, m, r, dst_nb[r]),), POISON_BYTE, dtype=torch.uint8).pin_memory()
             for r in range(nd)]
    torch.cuda.synchronize()
    sums = [int(t.view(torch.int64).sum().item()) for t in h_src]
    dbt, total, up, down = remp.remp_reshard_host(S, D, m, w.seq_lens, w.block_tables, h_src, src_nb, h_dst, dst_nb)
    want_dbt, _off, want_total = orc.alloc(w.seq_lens, w.max_blocks_per_seq, m.block_size, 0, dst_nb)
    assert total == want_total == w.live_blocks and np.array_equal(dbt, want_dbt)
    r_bytes = total * L * 2 * m.num_kv_heads * m.block_size * m.head_dim * m.elem_bytes
    assert up == r_bytes + w.seq_lens.size * 4 + w.block_tables.size * 4       # only live blocks were read
    for l in range(L):
        ps, pd = orc.pp_owner(S, L, l), orc.pp_owner(D, L, l)
        cur = []
        for t in range(S.tp):
            r = orc.rank_of(S, ps, t)
            lb = orc.layer_slab_bytes(S, m, src_nb[r])
            o = (l - orc.stage_first(S, L, ps)) * lb
            cur.append(h_src[r][o:o + lb].numpy())
        nbD = [dst_nb[orc.rank_of(D, pd, t)] for t in range(D.tp)]
        nxt = [np.full(orc.layer_slab_bytes(D, m, nbD[t]), POISON_BYTE, dtype=np.uint8) for t in range(D.tp)]
        assert orc.migrate_layer(S, D, m, w.seq_lens, w.block_tables, want_dbt, cur,
                                 [src_nb[orc.rank_of(S, ps, t)] for t in range(S.tp)], nxt, nbD) == 0
        for t in range(D.tp):
            r = orc.rank_of(D, pd, t)
            lb = orc.layer_slab_bytes(D, m, nbD[t])
            o = (l - orc.stage_first(D, L, pd)) * lb
            assert np.array_equal(h_dst[r][o:o + lb].numpy(), nxt[t]), (l, t)
    assert [int(t.view(torch.int64).sum().item()) for t in h_src] == sums
