"""CPU-only checks of the C-ABI library: it loads, exports what include/remp.h declares, and its host
planner (topology maps + Algorithm 1) agrees with the oracle. No kernel runs here."""
import os
import re

import numpy as np
import pytest
import torch

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from paper_2606_18741_b200 import _lib
from paper_2606_18741_b200.synth import Shape, Topo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = _lib.load()
    header = open(os.path.join(ROOT, "include", "remp.h")).read()
    declared = set(re.findall(r"\b(remp_[a-z_]+)\s*\(", header))
    assert declared == set(_lib.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def _fake_tables(n=3, maxb=4):
    # plan creation reads no device memory, so CPU tensors posing as device pointers are safe here
    class T:  # minimal stand-in with the attributes the binding marshals
        def __init__(self, t): self.t = t
        is_cuda = True
        def is_contiguous(self): return True
        @property
        def shape(self): return self.t.shape
        @property
        def dtype(self): return self.t.dtype
        def dim(self): return self.t.dim()
        def data_ptr(self): return self.t.data_ptr()
    return T(torch.zeros(n, dtype=torch.int32)), T(torch.zeros(n, maxb, dtype=torch.int32))


MODELS = [(32, 32), (80, 8), (64, 8), (48, 4), (6, 4), (7, 2)]
LAYOUTS = [Topo(8, 1), Topo(4, 2), Topo(2, 4), Topo(1, 8), Topo(4, 1), Topo(2, 2), Topo(1, 4), Topo(16, 1),
           Topo(2, 3, None)]


def test_plan_items_equal_oracle_items():
    lens, bt = _fake_tables()
    for (L, H) in MODELS:
        m = Shape(L, H, 128, 16, 2)
        for S in LAYOUTS:
            for D in LAYOUTS:
                legal = orc.topo_check(S, m) == 0 and orc.topo_check(D, m) == 0
                if not legal:
                    with pytest.raises(remp.RempError) as ei:
                        remp.remp_plan_create(S, D, m, lens, bt)
                    assert ei.value.status == remp.REMP_ERR_INVALID_TOPOLOGY
                    continue
                plan = remp.remp_plan_create(S, D, m, lens, bt)
                got = remp.remp_plan_get_items(plan)
                remp.remp_plan_destroy(plan)
                want = orc.plan(S, D, m)
                assert got.shape == want.shape, (L, H, str(S), str(D))
                assert sorted(map(tuple, got)) == sorted(map(tuple, want))


def test_explicit_stage_boundaries_and_shard_bytes():
    m = Shape(7, 2, 8, 4, 2)
    S = Topo(2, 3, (0, 1, 5, 7))
    for r in range(6):
        assert remp.remp_shard_bytes(S, m, r, 9) == orc.shard_bytes(S, m, r, 9)
    for (L, H) in MODELS:
        m = Shape(L, H, 64, 16, 1)
        for T in LAYOUTS:
            if orc.topo_check(T, m):
                continue
            for r in range(T.tp * T.pp):
                assert remp.remp_shard_bytes(T, m, r, 5) == orc.shard_bytes(T, m, r, 5)
    with pytest.raises(remp.RempError):
        remp.remp_shard_bytes(Topo(2, 3, (0, 5, 5, 7)), Shape(7, 2, 8, 4, 2), 0, 1)


def test_shape_and_argument_errors():
    lens, bt = _fake_tables()
    with pytest.raises(remp.RempError) as ei:
        remp.remp_plan_create(Topo(1, 1), Topo(1, 1), Shape(2, 2, 3, 1, 2), lens, bt)     # 6-byte head slice
    assert ei.value.status == remp.REMP_ERR_SHAPE
    with pytest.raises(remp.RempError) as ei:
        remp.remp_plan_create(Topo(1, 1), Topo(1, 1), Shape(2, 2, 8, 4, 3), lens, bt)
    assert ei.value.status == remp.REMP_ERR_SHAPE
    plan = remp.remp_plan_create(Topo(1, 1), Topo(2, 1), Shape(2, 2, 8, 4, 2), lens, bt)
    r, w = remp.remp_plan_traffic(plan, 10)
    assert r == 10 * 2 * 2 * 2 * 4 * 8 * 2 and w == r
    with pytest.raises(remp.RempError) as ei:
        remp.remp_plan_set_option(plan, 99, 1)
    assert ei.value.status == remp.REMP_ERR_INVALID_ARG
    assert remp.remp_plan_status(plan, 0) == remp.REMP_OK      # nothing has run on a device
    remp.remp_plan_destroy(plan)
    plan = remp.remp_plan_create(Topo(1, 1), Topo(4, 1), Shape(2, 2, 8, 4, 2), lens, bt)   # replication 2
    r, w = remp.remp_plan_traffic(plan, 10)
    assert w == 2 * r
    remp.remp_plan_destroy(plan)


def test_header_is_plain_c_and_planner_runs_from_c(tmp_path):
    """Compile a C program against include/remp.h with gcc -std=c99 -pedantic and run it against libremp.so."""
    import subprocess
    exe = tmp_path / "c_abi_check"
    lib_dir = os.path.dirname(_lib.LIB_PATH)
    _lib.load()
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c_abi_check.c"), "-o", str(exe), "-L", lib_dir, "-l:libremp.so",
                    f"-Wl,-rpath,{lib_dir}", "-Wl,-rpath,/usr/local/cuda/lib64"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stdout, out.stderr)
    assert "c abi ok: 640 items" in out.stdout


def test_planner_equals_oracle_on_random_topologies_with_explicit_stages():
    """Random legal topology pairs with explicit uneven stage boundaries: item lists equal as multisets and
    shard sizes agree for every rank."""
    rng = np.random.default_rng(99)
    lens, bt = _fake_tables()
    for _ in range(300):
        L = int(rng.integers(1, 25))
        Hh = int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 32]))
        m = Shape(L, Hh, 64, 16, 2)

        def topo():
            tps = [t for t in (1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64) if (Hh % t == 0 if t <= Hh else t % Hh == 0)]
            tp = int(rng.choice(tps))
            pp = int(rng.integers(1, min(L, 8) + 1))
            if pp > 1 and rng.random() < 0.5:
                cuts = sorted(rng.choice(np.arange(1, L), size=pp - 1, replace=False).tolist())
                return Topo(tp, pp, tuple([0] + cuts + [L]))
            return Topo(tp, pp)

        S, D = topo(), topo()
        assert orc.topo_check(S, m) == 0 and orc.topo_check(D, m) == 0
        plan = remp.remp_plan_create(S, D, m, lens, bt)
        got = remp.remp_plan_get_items(plan)
        remp.remp_plan_destroy(plan)
        want = orc.plan(S, D, m)
        assert sorted(map(tuple, got)) == sorted(map(tuple, want)), (L, Hh, S, D)
        for T in (S, D):
            for r in range(T.tp * T.pp):
                assert remp.remp_shard_bytes(T, m, r, 7) == orc.shard_bytes(T, m, r, 7)


def test_partition_equals_oracle_partition():
    """remp_plan_partition against the oracle's per-device view of the plan (host only)."""
    lens, bt = _fake_tables()
    rng = np.random.default_rng(5)
    for (L, H) in ((80, 8), (32, 32), (6, 4)):
        m = Shape(L, H, 128, 16, 2)
        legal = [T for T in LAYOUTS if orc.topo_check(T, m) == 0]
        for S in legal:
            for D in legal:
                ndev = int(rng.integers(1, 5))
                sdev = [int(x) for x in rng.integers(0, ndev, size=S.tp * S.pp)]
                ddev = [int(x) for x in rng.integers(0, ndev, size=D.tp * D.pp)]
                plan = remp.remp_plan_create(S, D, m, lens, bt)
                try:
                    for q in range(ndev):
                        got_r, got_s = remp.remp_plan_partition(plan, sdev, ddev, q)
                        want_r, want_s = orc.plan_partition(S, D, m, sdev, ddev, q)
                        assert sorted(map(tuple, got_r)) == sorted(map(tuple, want_r))
                        assert sorted(map(tuple, got_s)) == sorted(map(tuple, want_s))
                finally:
                    remp.remp_plan_destroy(plan)
