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
