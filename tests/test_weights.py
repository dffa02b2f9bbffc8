"""Model weights from a host store (section 3.3): the packed shard layout (host only) and, on a GPU, the shards
themselves against numpy slicing of the full tensors, for the paper's four model shapes and seven layouts at
reduced width."""
import os

import numpy as np
import pytest

import paper_2606_18741_b200 as remp
from oracle import remp_oracle as orc
from paper_2606_18741_b200.synth import Topo, weight_store

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
PART = {"replicated": remp.REMP_W_REPLICATED, "rows": remp.REMP_W_SPLIT_ROWS, "cols": remp.REMP_W_SPLIT_COLS,
        "row_groups": remp.REMP_W_SPLIT_ROW_GROUPS}
SCOPE = {"layer": remp.REMP_W_EVERY_LAYER, "first": remp.REMP_W_FIRST_STAGE, "last": remp.REMP_W_LAST_STAGE}


def _models():
    rows = [l.split() for l in open(os.path.join(GOLD, "model_widths.txt")) if l.strip() and l[0] != "#"]
    return [(n, int(a), int(b), int(c), int(d)) for n, a, b, c, d in rows]


def _layouts():
    rows = [l.split() for l in open(os.path.join(GOLD, "layouts.txt")) if l.strip() and l[0] != "#"]
    return [Topo(int(a), int(b)) for a, b in rows]


def _c_params(store, tensors=None):
    return remp.make_weight_params([{"tensor": (tensors[i] if tensors else p["tensor"]), "partition": PART[p["partition"]],
                                     "scope": SCOPE[p["scope"]], "groups": p["groups"]} for i, p in enumerate(store)])


def _small_store(name, L, hidden, heads, kv, layers=None):
    # reduced width: head_dim 8, hidden = 8 * heads; a few layers stand for all (the stage map is checked apart)
    return weight_store(layers or L, hidden, heads, kv, seed=len(name), scale=hidden // (8 * heads), vocab=256)


# ---------------------------------------------------------------- oracle pins (numpy only)

def test_weight_slices_of_all_ranks_reassemble_the_full_tensors():
    """TP slices concatenated along their split axis give the tensor back; replicated group slices equal the group
    of the lowest owner; every layer is held by exactly one stage; first/last-stage tensors by that stage only."""
    L = 5
    store = weight_store(L, 64, 8, 2, seed=1, scale=1, vocab=64)
    for T in [Topo(1, 1), Topo(2, 1), Topo(4, 2), Topo(8, 5), Topo(2, 3), Topo(1, 4)]:
        for p in store:
            per_rank = [orc.weight_slice(T, L, r, p["tensor"], p["partition"], p["scope"], p["groups"])
                        for r in range(T.tp * T.pp)]
            if p["scope"] == "layer":
                held = sorted(l for stage in range(T.pp) for l in per_rank[stage * T.tp])
                assert held == list(range(L))
                keys = [(stage, l) for stage in range(T.pp) for l in per_rank[stage * T.tp]]
            else:
                stage = 0 if p["scope"] == "first" else T.pp - 1
                assert all(bool(per_rank[r]) == (r // T.tp == stage) for r in range(T.tp * T.pp))
                keys = [(stage, -1)]
            for stage, l in keys:
                full = p["tensor"][l] if l >= 0 else p["tensor"]
                parts = [per_rank[stage * T.tp + t][l] for t in range(T.tp)]
                if p["partition"] == "replicated":
                    assert all(np.array_equal(x, full) for x in parts)
                elif p["partition"] == "rows":
                    assert np.array_equal(np.concatenate(parts, axis=0), full)
                elif p["partition"] == "cols":
                    assert np.array_equal(np.concatenate(parts, axis=1), full)
                else:
                    G = p["groups"]
                    rep = max(1, T.tp // G)
                    assert np.array_equal(np.concatenate(parts[::rep], axis=0), full)      # one owner per group
                    for t in range(T.tp):
                        assert np.array_equal(parts[t], parts[t - t % rep])                # replicas are equal


# ---------------------------------------------------------------- packed layout (library, host only)

@pytest.mark.parametrize("name,L,hidden,heads,kv", _models())
def test_packed_layout_matches_the_oracle_slices(name, L, hidden, heads, kv):
    store = _small_store(name, L, hidden, heads, kv, layers=1)        # one stored layer: only shapes are used here
    tensors = [np.broadcast_to(p["tensor"], (L,) + p["tensor"].shape[1:]) if p["scope"] == "layer" else p["tensor"]
               for p in store]                                         # all L layers without L copies
    cp = remp.make_weight_params([{"tensor": np.ascontiguousarray(p["tensor"]), "partition": PART[p["partition"]],
                                   "scope": SCOPE[p["scope"]], "groups": p["groups"]} for p in store])
    for i, p in enumerate(store):                                      # layer stride 0 would be refused: one instance each
        if p["scope"] == "layer":
            cp[i].layer_stride = p["tensor"][0].nbytes
    for T in _layouts():
        if kv % T.tp and T.tp % kv:
            continue
        for rank in range(T.tp * T.pp):
            spans = []
            for i, p in enumerate(store):
                want = orc.weight_slice(T, L, rank, tensors[i], p["partition"], p["scope"], p["groups"])
                for l, a in want.items():
                    off, rows, cols = remp.remp_weight_slice(T, L, cp, rank, i, max(l, 0))
                    assert (rows, cols) == a.shape and off % 256 == 0, (name, str(T), rank, p["name"], l)
                    spans.append((off, off + a.nbytes))
                if not want:
                    with pytest.raises(remp.RempError):
                        remp.remp_weight_slice(T, L, cp, rank, i, 0)
            spans.sort()
            assert spans[0][0] == 0 and all(b <= c for (_a, b), (c, _d) in zip(spans, spans[1:]))     # disjoint, packed
            total = remp.remp_weight_shard_bytes(T, L, cp, rank)
            assert spans[-1][1] <= total < spans[-1][1] + 256


def test_weight_store_errors():
    store = weight_store(2, 64, 8, 2, seed=0, vocab=64)
    cp = _c_params(store)
    with pytest.raises(remp.RempError) as ei:                          # 3 does not divide the 8 x 8 q rows
        remp.remp_weight_shard_bytes(Topo(3, 1), 2, cp, 0)
    assert ei.value.status == remp.REMP_ERR_INVALID_TOPOLOGY
    with pytest.raises(remp.RempError) as ei:                          # more stages than layers
        remp.remp_weight_shard_bytes(Topo(1, 3), 2, cp, 0)
    assert ei.value.status == remp.REMP_ERR_INVALID_TOPOLOGY
    with pytest.raises(remp.RempError) as ei:
        remp.remp_weight_shard_bytes(Topo(2, 1), 2, cp, 2)
    assert ei.value.status == remp.REMP_ERR_INVALID_ARG
    odd = [{"tensor": np.zeros((2, 4, 12), dtype=np.uint16), "partition": remp.REMP_W_SPLIT_COLS,
            "scope": remp.REMP_W_EVERY_LAYER, "groups": 0}]           # 12 columns over TP2: 12-byte row slices
    with pytest.raises(remp.RempError) as ei:
        remp.remp_weight_shard_bytes(Topo(2, 1), 2, remp.make_weight_params(odd), 0)
    assert ei.value.status == remp.REMP_ERR_SHAPE


# ---------------------------------------------------------------- the shards themselves (GPU)

@pytest.mark.gpu
@pytest.mark.parametrize("pinned,max_ctas", [(True, 0), (False, 0), (True, 3)])
@pytest.mark.parametrize("name,L,hidden,heads,kv", _models())
def test_shards_equal_numpy_slices_of_the_store(name, L, hidden, heads, kv, pinned, max_ctas):
    """Every target rank's shard, rebuilt from the host store by the gather kernel (page-locked store; also with
    its grid bounded to a few thread blocks) or the copy engine (pageable store), holds exactly the numpy slices
    of the full tensors; padding keeps its bytes."""
    import torch
    Lr = 6                                                              # six layers stand for the model's depth
    store = _small_store(name, L, hidden, heads, kv, layers=Lr)
    host = []
    for p in store:
        t = torch.from_numpy(p["tensor"].view(np.int16))               # torch has no uint16: same bytes
        host.append(t.pin_memory() if pinned else t.clone())
    cp = _c_params(store, host)
    for T in _layouts() + [Topo(16, 1), Topo(2, 3)]:
        if (kv % T.tp and T.tp % kv) or T.pp > Lr or (8 * heads) % (8 * T.tp):
            continue                    # needs whole KV-head groups, enough layers, and 16-byte rows in every column slice
        nr = T.tp * T.pp
        sizes = [remp.remp_weight_shard_bytes(T, Lr, cp, r) for r in range(nr)]
        shards = [torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda") for n in sizes]
        moved = remp.remp_weights_reshard(T, Lr, cp, shards, max_ctas=max_ctas)
        torch.cuda.synchronize()
        got = [s.cpu().numpy() for s in shards]
        want_bytes = 0
        for r in range(nr):
            covered = np.zeros(sizes[r], dtype=bool)
            for i, p in enumerate(store):
                for l, a in orc.weight_slice(T, Lr, r, p["tensor"], p["partition"], p["scope"], p["groups"]).items():
                    off, rows, cols = remp.remp_weight_slice(T, Lr, cp, r, i, max(l, 0))
                    flat = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
                    assert np.array_equal(got[r][off:off + flat.size], flat), (name, str(T), r, p["name"], l)
                    covered[off:off + flat.size] = True
                    want_bytes += flat.size
            assert (got[r][~covered] == 0x5A).all()                     # padding untouched
        assert moved == want_bytes


@pytest.mark.gpu
def test_store_in_registered_host_memory_is_gathered_by_the_kernel():
    """A store that lives in ordinary host memory page-locked after the fact (cudaHostRegister, as a shared-memory
    weight store would be) takes the gather-kernel path like one allocated page-locked: same shards, one launch."""
    import torch
    name, L, hidden, heads, kv = _models()[1]
    Lr = 4
    store = _small_store(name, L, hidden, heads, kv, layers=Lr)
    rt = torch.cuda.cudart()
    host = [np.ascontiguousarray(p["tensor"]).copy() for p in store]
    registered = []
    try:
        for a in host:
            rc = rt.cudaHostRegister(a.ctypes.data, a.nbytes, 0)
            assert int(rc) == 0, rc
            registered.append(a)
        cp = _c_params(store, [torch.from_numpy(a.view(np.int16)) for a in host])
        T = Topo(4, 2)
        nr = T.tp * T.pp
        sizes = [remp.remp_weight_shard_bytes(T, Lr, cp, r) for r in range(nr)]
        shards = [torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda") for n in sizes]
        before = remp.remp_kernel_launch_count()
        remp.remp_weights_reshard(T, Lr, cp, shards)
        torch.cuda.synchronize()
        assert remp.remp_kernel_launch_count() - before == 1          # the gather kernel, not per-slice copies
        for r in range(nr):
            got = shards[r].cpu().numpy()
            for i, p in enumerate(store):
                for l, a in orc.weight_slice(T, Lr, r, p["tensor"], p["partition"], p["scope"], p["groups"]).items():
                    off, _rows, _cols = remp.remp_weight_slice(T, Lr, cp, r, i, max(l, 0))
                    flat = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
                    assert np.array_equal(got[off:off + flat.size], flat), (r, p["name"], l)
    finally:
        for a in registered:
            rt.cudaHostUnregister(a.ctypes.data)
