"""ctypes front end of the C oracle (oracle/remp_oracle.c). TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; the CUDA
library never does. Topologies and shapes are duck-typed (.tp/.pp/.layer_start and
.num_layers/.num_kv_heads/.head_dim/.block_size/.elem_bytes).
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

_lib = None


class _Topo(C.Structure):
    _fields_ = [("tp", C.c_int32), ("pp", C.c_int32), ("layer_start", C.POINTER(C.c_int32))]


class _Shape(C.Structure):
    _fields_ = [("L", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("bs", C.c_int32), ("e", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        P = C.POINTER
        L.orc_stage_first.argtypes = [P(_Topo), C.c_int, C.c_int]
        L.orc_pp_owner.argtypes = [P(_Topo), C.c_int, C.c_int]
        for f in ("orc_rep", "orc_heads_per_rank"):
            getattr(L, f).argtypes = [P(_Topo), C.c_int]
        for f in ("orc_head_lo", "orc_head_hi", "orc_tp_owner"):
            getattr(L, f).argtypes = [P(_Topo), C.c_int, C.c_int]
        L.orc_owns_head.argtypes = [P(_Topo), C.c_int, C.c_int, C.c_int]
        L.orc_rank.argtypes = [P(_Topo), C.c_int, C.c_int]
        L.orc_topo_check.argtypes = [P(_Topo), P(_Shape)]
        L.orc_head_slice_bytes.argtypes = [P(_Shape)]
        L.orc_head_slice_bytes.restype = C.c_int64
        L.orc_layer_slab_bytes.argtypes = [P(_Topo), P(_Shape), C.c_int64]
        L.orc_layer_slab_bytes.restype = C.c_int64
        L.orc_shard_bytes.argtypes = [P(_Topo), P(_Shape), C.c_int, C.c_int64]
        L.orc_shard_bytes.restype = C.c_int64
        L.orc_offset.argtypes = [P(_Topo), P(_Shape), C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int64, C.c_int,
                                 C.c_int, C.c_int]
        L.orc_offset.restype = C.c_int64
        L.orc_alloc.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int, C.c_void_p,
                                C.c_void_p]
        L.orc_alloc.restype = C.c_int64
        L.orc_alloc_preempt.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int,
                                        C.c_void_p, C.c_void_p]
        L.orc_alloc_preempt.restype = C.c_int64
        L.orc_alloc_shared.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int64,
                                       C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_alloc_shared.restype = C.c_int64
        L.orc_plan.argtypes = [P(_Topo), P(_Topo), P(_Shape), C.c_int, C.c_void_p, C.c_int]
        L.orc_migrate_layer.argtypes = [P(_Topo), P(_Topo), P(_Shape), C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                        C.c_int]
        L.orc_migrate.argtypes = [P(_Topo), P(_Topo), P(_Shape), C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                  C.c_int, C.c_int]
        L.orc_migrate_layout.argtypes = L.orc_migrate.argtypes + [C.c_int, C.c_int]
        L.orc_migrate_layer_layout.argtypes = L.orc_migrate_layer.argtypes + [C.c_int, C.c_int]
        L.orc_migrate_ex.argtypes = L.orc_migrate.argtypes + [C.c_int, C.c_int, C.c_int]
        _lib = L
    return _lib


class CapacityError(Exception):
    pass


def _topo(T):
    """Returns (struct, keepalive)."""
    ls = getattr(T, "layer_start", None)
    if ls is None:
        return _Topo(T.tp, T.pp, None), None
    arr = (C.c_int32 * len(ls))(*ls)
    return _Topo(T.tp, T.pp, C.cast(arr, C.POINTER(C.c_int32))), arr


def _shape(m):
    return _Shape(m.num_layers, m.num_kv_heads, m.head_dim, m.block_size, m.elem_bytes)


def topo_check(T, m) -> int:
    t, _k = _topo(T)
    return lib().orc_topo_check(C.byref(t), C.byref(_shape(m)))


def num_ranks(T) -> int:
    return T.tp * T.pp


def stage_first(T, L: int, p: int) -> int:
    t, _k = _topo(T)
    return lib().orc_stage_first(C.byref(t), L, p)


def pp_owner(T, L: int, l: int) -> int:
    t, _k = _topo(T)
    return lib().orc_pp_owner(C.byref(t), L, l)


def rep(T, H: int) -> int:
    t, _k = _topo(T)
    return lib().orc_rep(C.byref(t), H)


def heads_per_rank(T, H: int) -> int:
    t, _k = _topo(T)
    return lib().orc_heads_per_rank(C.byref(t), H)


def head_range(T, H: int, tp_rank: int):
    t, _k = _topo(T)
    return lib().orc_head_lo(C.byref(t), H, tp_rank), lib().orc_head_hi(C.byref(t), H, tp_rank)


def owns_head(T, H: int, tp_rank: int, h: int) -> bool:
    t, _k = _topo(T)
    return bool(lib().orc_owns_head(C.byref(t), H, tp_rank, h))


def tp_owner(T, H: int, h: int) -> int:
    t, _k = _topo(T)
    return lib().orc_tp_owner(C.byref(t), H, h)


def rank_of(T, p: int, tpr: int) -> int:
    t, _k = _topo(T)
    return lib().orc_rank(C.byref(t), p, tpr)


def head_slice_bytes(m) -> int:
    return lib().orc_head_slice_bytes(C.byref(_shape(m)))


def layer_slab_bytes(T, m, nb: int) -> int:
    t, _k = _topo(T)
    return lib().orc_layer_slab_bytes(C.byref(t), C.byref(_shape(m)), nb)


def shard_bytes(T, m, rank: int, nb: int) -> int:
    t, _k = _topo(T)
    return lib().orc_shard_bytes(C.byref(t), C.byref(_shape(m)), rank, nb)


def offset(T, m, rank: int, nb: int, l: int, kv: int, blk: int, h: int, tok: int = 0, dim: int = 0) -> int:
    t, _k = _topo(T)
    return lib().orc_offset(C.byref(t), C.byref(_shape(m)), rank, nb, l, kv, blk, h, tok, dim)


def alloc(seq_lens: np.ndarray, max_blocks: int, block_size: int, base: int, caps: Sequence[int]):
    """Serial allocator. Returns (dst_block_tables int32 [n][max_blocks], off int32 [n+1], total)."""
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    n = lens.shape[0]
    capa = np.ascontiguousarray(caps, dtype=np.int64)
    dst_bt = np.full((n, max_blocks), -7, dtype=np.int32)
    off = np.zeros(n + 1, dtype=np.int32)
    total = lib().orc_alloc(n, max_blocks, lens.ctypes.data, block_size, base, capa.ctypes.data, len(capa),
                            dst_bt.ctypes.data, off.ctypes.data)
    if total == -1:
        raise CapacityError("live blocks exceed a destination pool")
    if total < 0:
        raise ValueError("a sequence needs more blocks than the table is wide")
    return dst_bt, off, int(total)


def alloc_preempt(seq_lens: np.ndarray, max_blocks: int, block_size: int, base: int, caps: Sequence[int]):
    """Capacity-constrained allocator: keeps the longest prefix of sequences that fits.
    Returns (dst_block_tables, preempted int32 [n], total blocks of the kept sequences)."""
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    n = lens.shape[0]
    capa = np.ascontiguousarray(caps, dtype=np.int64)
    dst_bt = np.full((n, max_blocks), -7, dtype=np.int32)
    pre = np.full(n, -7, dtype=np.int32)
    total = lib().orc_alloc_preempt(n, max_blocks, lens.ctypes.data, block_size, base, capa.ctypes.data, len(capa),
                                    dst_bt.ctypes.data, pre.ctypes.data)
    if total < 0:
        raise ValueError("a sequence needs more blocks than the table is wide")
    return dst_bt, pre, int(total)


def alloc_shared(seq_lens: np.ndarray, block_tables: np.ndarray, block_size: int, base: int, src_pool: int,
                 caps: Sequence[int]):
    """Sharing-preserving allocator: equal source blocks get equal destination blocks.
    Returns (dst_block_tables, blocks allocated, bad-id flag)."""
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    capa = np.ascontiguousarray(caps, dtype=np.int64)
    dst_bt = np.full(bt.shape, -7, dtype=np.int32)
    bad = C.c_int32(0)
    total = lib().orc_alloc_shared(lens.shape[0], bt.shape[1], lens.ctypes.data, bt.ctypes.data, block_size, base,
                                   src_pool, capa.ctypes.data, len(capa), dst_bt.ctypes.data, C.byref(bad))
    if total == -1:
        raise CapacityError("distinct live blocks exceed a destination pool")
    if total < 0:
        raise ValueError("a sequence needs more blocks than the table is wide")
    return dst_bt, int(total), bool(bad.value)


def plan(S, D, m, dedupe: bool = True) -> np.ndarray:
    """Algorithm 1 items, int32 [n][5] = (src rank, dst rank, layer, h_lo, h_hi)."""
    s, _ks = _topo(S)
    d, _kd = _topo(D)
    sh = _shape(m)
    n = lib().orc_plan(C.byref(s), C.byref(d), C.byref(sh), int(dedupe), None, 0)
    items = np.zeros((n, 5), dtype=np.int32)
    lib().orc_plan(C.byref(s), C.byref(d), C.byref(sh), int(dedupe), items.ctypes.data, n)
    return items


def plan_partition(S, D, m, src_rank_device: Sequence[int], dst_rank_device: Sequence[int], device: int):
    """The plan seen from one device when the ranks are spread over several (section 3.4.2: the send side mirrors
    the receive side; section 3.4.3: an item is a local copy when both ranks share a device, a remote transfer
    otherwise). Returns (recv, send): recv = the items whose destination rank is on `device`, rows
    (src rank, dst rank, layer, h_lo, h_hi, device of the src rank); send = the items whose source rank is on
    `device` and whose destination rank is elsewhere, 6th column = device of the dst rank."""
    items = plan(S, D, m, dedupe=True)
    sd = np.asarray(src_rank_device, dtype=np.int32)[items[:, 0]]
    dd = np.asarray(dst_rank_device, dtype=np.int32)[items[:, 1]]
    recv = np.concatenate([items[dd == device], sd[dd == device, None]], axis=1)
    out = (sd == device) & (dd != device)
    send = np.concatenate([items[out], dd[out, None]], axis=1)
    return recv.astype(np.int32), send.astype(np.int32)


def _ptr_array(bufs: Sequence[np.ndarray]):
    for b in bufs:
        assert b.dtype == np.uint8 and b.flags["C_CONTIGUOUS"]
    return (C.c_void_p * len(bufs))(*[b.ctypes.data for b in bufs])


def migrate(S, D, m, seq_lens, block_tables, dst_block_tables, src: List[np.ndarray], src_nb: Sequence[int],
            dst: List[np.ndarray], dst_nb: Sequence[int], mode: str = "row", nthreads: int = 1,
            layer_lo: int = 0, layer_hi: Optional[int] = None, src_layout: str = "head", dst_layout: str = "head",
            valid_only: bool = False) -> int:
    """Re-shard src (one uint8 array per source rank) into dst (one per destination rank, in place).
    Layouts: "head" = [block][head][token][dim] (canonical), "token" = [block][token][head][dim]."""
    s, _ks = _topo(S)
    d, _kd = _topo(D)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    dbt = np.ascontiguousarray(dst_block_tables, dtype=np.int32)
    assert bt.shape == dbt.shape and bt.shape[0] == lens.shape[0]
    snb = np.ascontiguousarray(src_nb, dtype=np.int64)
    dnb = np.ascontiguousarray(dst_nb, dtype=np.int64)
    assert len(src) == S.tp * S.pp and len(dst) == D.tp * D.pp
    for r, b in enumerate(src):
        assert b.size == shard_bytes(S, m, r, int(snb[r]))
    for r, b in enumerate(dst):
        assert b.size == shard_bytes(D, m, r, int(dnb[r]))
    sp, dp = _ptr_array(src), _ptr_array(dst)
    hi = m.num_layers if layer_hi is None else layer_hi
    lay = {"head": 0, "token": 1}
    return lib().orc_migrate_ex(C.byref(s), C.byref(d), C.byref(_shape(m)), lens.shape[0], bt.shape[1],
                                lens.ctypes.data, bt.ctypes.data, dbt.ctypes.data, sp, snb.ctypes.data, dp,
                                dnb.ctypes.data, {"elem": 0, "row": 1}[mode], nthreads, layer_lo, hi,
                                lay[src_layout], lay[dst_layout], int(valid_only))


def migrate_layer(S, D, m, seq_lens, block_tables, dst_block_tables, src_slabs: List[np.ndarray],
                  src_nb: Sequence[int], dst_slabs: List[np.ndarray], dst_nb: Sequence[int], mode: str = "row",
                  src_layout: str = "head", dst_layout: str = "head") -> int:
    """One layer: src_slabs[t] is that layer's slab on source TP rank t of the stage that owns it,
    dst_slabs[t] likewise on the destination side (modified in place)."""
    s, _ks = _topo(S)
    d, _kd = _topo(D)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    dbt = np.ascontiguousarray(dst_block_tables, dtype=np.int32)
    snb = np.ascontiguousarray(src_nb, dtype=np.int64)
    dnb = np.ascontiguousarray(dst_nb, dtype=np.int64)
    assert len(src_slabs) == S.tp and len(dst_slabs) == D.tp
    for t, b in enumerate(src_slabs):
        assert b.size == layer_slab_bytes(S, m, int(snb[t]))
    for t, b in enumerate(dst_slabs):
        assert b.size == layer_slab_bytes(D, m, int(dnb[t]))
    sp, dp = _ptr_array(src_slabs), _ptr_array(dst_slabs)
    lay = {"head": 0, "token": 1}
    return lib().orc_migrate_layer_layout(C.byref(s), C.byref(d), C.byref(_shape(m)), lens.shape[0], bt.shape[1],
                                          lens.ctypes.data, bt.ctypes.data, dbt.ctypes.data, sp, snb.ctypes.data, dp,
                                          dnb.ctypes.data, 0, D.tp, {"elem": 0, "row": 1}[mode], lay[src_layout],
                                          lay[dst_layout])


# ---------------------------------------------------------------- model weights from a host store (section 3.3)

def weight_slice(T, num_layers: int, rank: int, tensor: np.ndarray, partition: str, scope: str = "layer",
                 groups: int = 0):
    """What target rank `rank` of topology T holds of one parameter of the full model state: PP selects the
    layers of the rank's stage, TP slices partitioned tensors, replicated ones are taken whole.
    tensor: [layers][rows][cols] for scope "layer", else [rows][cols] (scope "first" / "last": only ranks of the
    first / last stage hold it). partition: "replicated", "rows" (dim 0 split evenly), "cols" (dim 1 split evenly),
    "row_groups" (dim 0 is `groups` equal groups dealt to TP ranks like KV heads).
    Returns {layer or -1: 2-D array}; numpy slicing only."""
    p, t = divmod(rank, T.tp)

    def tp_part(a):
        if partition == "replicated":
            return a
        if partition == "rows":
            return np.split(a, T.tp, axis=0)[t]
        if partition == "cols":
            return np.split(a, T.tp, axis=1)[t]
        lo, hi = head_range(T, groups, t)                      # the oracle's own tp_owner, on row groups
        g = a.reshape(groups, a.shape[0] // groups, a.shape[1])
        return g[lo:hi].reshape(-1, a.shape[1])

    if scope == "layer":
        return {l: tp_part(tensor[l]) for l in range(stage_first(T, num_layers, p), stage_first(T, num_layers, p + 1))}
    if (scope == "first" and p == 0) or (scope == "last" and p == T.pp - 1):
        return {-1: tp_part(tensor)}
    return {}
