"""Property-based pins of the oracle (hypothesis): for random model shapes, topology pairs, stage boundaries,
tables, base offsets and pool sizes the C oracle equals the numpy slicing statement of the result, the
source-driven enumerator finds every row exactly once per replica, and the plan has its closed-form size."""
import math

import numpy as np
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import brute
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import Shape, Topo
from tests import helpers as H


@st.composite
def topo_for(draw, L, Hh):
    tps = [t for t in (1, 2, 3, 4, 6, 8, 12, 16) if (Hh % t == 0 if t <= Hh else t % Hh == 0)]
    tp = draw(st.sampled_from(tps))
    pp = draw(st.integers(1, min(L, 4)))
    if pp > 1 and draw(st.booleans()):
        cuts = sorted(draw(st.lists(st.integers(1, L - 1), min_size=pp - 1, max_size=pp - 1, unique=True)))
        return Topo(tp, pp, tuple([0] + cuts + [L]))
    return Topo(tp, pp)


@st.composite
def case(draw):
    L = draw(st.integers(1, 6))
    Hh = draw(st.sampled_from([1, 2, 4, 6, 8]))
    m = Shape(L, Hh, draw(st.sampled_from([4, 8])), draw(st.sampled_from([1, 2, 4])), draw(st.sampled_from([1, 2, 4])))
    S, D = draw(topo_for(L, Hh)), draw(topo_for(L, Hh))
    n = draw(st.integers(0, 6))
    lens = np.array(draw(st.lists(st.integers(0, 5 * m.block_size), min_size=n, max_size=n)), dtype=np.int32)
    need = -(-lens.astype(np.int64) // m.block_size)
    total = int(need.sum())
    pool = total + draw(st.integers(0, 3)) + 1
    perm = np.random.default_rng(draw(st.integers(0, 2**31))).permutation(pool)[:total].astype(np.int32)
    maxb = int(need.max(initial=0)) + draw(st.integers(1, 2))
    bt = np.full((n, maxb), -1, dtype=np.int32)
    pos = 0
    for s in range(n):
        bt[s, :need[s]] = perm[pos:pos + need[s]]
        pos += need[s]
    base = draw(st.integers(0, 3))
    seed = draw(st.integers(0, 2**31))
    return m, S, D, lens, bt, pool, base, seed


@settings(max_examples=120, deadline=None, suppress_health_check=[HealthCheck.too_slow, HealthCheck.data_too_large])
@given(case())
def test_oracle_equals_slicing_and_is_exactly_once(c):
    m, S, D, lens, bt, pool, base, seed = c
    G = H.random_global(m, pool, seed)
    src = H.shards_from_global(S, m, G)
    ns, nd = S.tp * S.pp, D.tp * D.pp
    total = int((-(-lens.astype(np.int64) // m.block_size)).sum())
    nb = [base + total + (r % 2) for r in range(nd)]
    dbt, off, tot = orc.alloc(lens, bt.shape[1], m.block_size, base, nb)
    assert tot == total
    before = H.poison_like([orc.shard_bytes(D, m, r, nb[r]) for r in range(nd)])
    after = [b.copy() for b in before]
    assert orc.migrate(S, D, m, lens, bt, dbt, src, [pool] * ns, after, nb, mode="row") == 0
    want = H.expected_by_slicing(D, m, G, H.flat_live_ids(m, lens, bt), base, nb)
    for a, b in zip(after, want):
        assert np.array_equal(a, b)
    res = brute.enumerate_check(S, D, m, lens, bt, dbt, src, [pool] * ns, after, nb, before)
    assert not any(res.values()), res
    # Algorithm 1: closed-form size
    a1, c1 = min(S.tp, m.num_kv_heads), min(D.tp, m.num_kv_heads)
    per_layer = D.tp if D.tp > m.num_kv_heads else a1 + c1 - math.gcd(a1, c1)
    assert len(orc.plan(S, D, m)) == m.num_layers * per_layer


@st.composite
def partition_case(draw):
    L = draw(st.integers(1, 6))
    Hh = draw(st.sampled_from([1, 2, 4, 6, 8]))
    m = Shape(L, Hh, 8, 4, 2)
    S, D = draw(topo_for(L, Hh)), draw(topo_for(L, Hh))
    ndev = draw(st.integers(1, 5))
    sdev = draw(st.lists(st.integers(0, ndev - 1), min_size=S.tp * S.pp, max_size=S.tp * S.pp))
    ddev = draw(st.lists(st.integers(0, ndev - 1), min_size=D.tp * D.pp, max_size=D.tp * D.pp))
    return m, S, D, ndev, sdev, ddev


@settings(max_examples=150, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(partition_case())
def test_partition_is_a_partition_with_mirrored_sends(c):
    """Any assignment of ranks to devices: the devices' receive lists partition the plan, the send lists are the
    remote receives regrouped by source device (section 3.4.2), and nothing is sent inside a device."""
    m, S, D, ndev, sdev, ddev = c
    items = sorted(map(tuple, orc.plan(S, D, m)))
    recv_all, send_all = [], []
    for q in range(ndev):
        recv, send = orc.plan_partition(S, D, m, sdev, ddev, q)
        assert all(ddev[r[1]] == q and r[5] == sdev[r[0]] for r in recv)
        assert all(sdev[r[0]] == q and r[5] == ddev[r[1]] and r[5] != q for r in send)
        recv_all += [tuple(r) for r in recv]
        send_all += [tuple(r[:5]) for r in send]
    assert sorted(r[:5] for r in recv_all) == items
    remote = sorted(r[:5] for r in recv_all if r[5] != ddev[r[1]])
    assert remote == sorted(send_all)


@st.composite
def weight_case(draw):
    L = draw(st.integers(1, 6))
    groups = draw(st.sampled_from([1, 2, 4, 8]))
    tp = draw(st.sampled_from([t for t in (1, 2, 4, 8, 16) if groups % t == 0 or t % groups == 0]))
    pp = draw(st.integers(1, L))
    rows = 16 * draw(st.integers(1, 3))          # divisible by every TP and group count drawn above
    cols = 16 * draw(st.integers(1, 3))
    partition = draw(st.sampled_from(["replicated", "rows", "cols", "row_groups"]))
    scope = draw(st.sampled_from(["layer", "first", "last"]))
    seed = draw(st.integers(0, 2**31))
    return L, groups, Topo(tp, pp), rows, cols, partition, scope, seed


@settings(max_examples=150, deadline=None)
@given(weight_case())
def test_weight_slices_tile_the_tensor(c):
    """Section 3.3: over all ranks every element of a parameter is held by exactly `replication` ranks - TP times
    for replicated tensors, TP/groups times when row groups are replicated, else once - and only by the stage
    that owns its layer (or the first / last stage)."""
    L, groups, T, rows, cols, partition, scope, _seed = c
    shape = (L, rows, cols) if scope == "layer" else (rows, cols)
    ids = np.arange(int(np.prod(shape)), dtype=np.int64).reshape(shape)      # every element names itself
    count = np.zeros(ids.size, dtype=np.int64)
    for r in range(T.tp * T.pp):
        for l, a in orc.weight_slice(T, L, r, ids, partition, scope, groups).items():
            if scope == "layer":
                assert orc.pp_owner(T, L, l) == r // T.tp                   # only the stage that owns the layer
                assert ((a // (rows * cols)) == l).all()
            np.add.at(count, a.reshape(-1), 1)
    want = T.tp if partition == "replicated" else (max(1, T.tp // groups) if partition == "row_groups" else 1)
    assert (count == want).all()

