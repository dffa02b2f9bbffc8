"""Thin Python binding of the C ABI in include/remp.h: argument marshalling only.

Function names match the C entry points. Device buffers are torch tensors (PyTorch is used for device
memory and streams only); every step of the path runs inside libremp's kernels.
"""
from __future__ import annotations

import ctypes as C
import functools
from typing import List, Optional, Sequence

import numpy as np

from . import _lib
from ._lib import RempBlockTables, RempHostShard, RempModelShape, RempShard, RempTopo, RempWeightParam

REMP_OK = 0
REMP_ERR_INVALID_ARG = -1
REMP_ERR_INVALID_TOPOLOGY = -2
REMP_ERR_SHAPE = -3
REMP_ERR_CAPACITY = -4
REMP_ERR_ALIAS = -5
REMP_ERR_BAD_BLOCK_ID = -6
REMP_ERR_STATE = -7
REMP_ERR_CUDA = -8
REMP_ERR_NOMEM = -9
REMP_ERR_BAD_LENGTH = -10

REMP_OPT_KERNEL = 1
REMP_OPT_CTAS_PER_SM = 2
REMP_OPT_CHUNK_BYTES = 3
REMP_OPT_VEC_BYTES = 4
REMP_OPT_TILE_ITEMS = 5
REMP_OPT_LANES_PER_WARP = 6
REMP_OPT_SCHEDULE = 7
REMP_OPT_VALID_TOKENS_ONLY = 8
REMP_OPT_ORDER = 9
REMP_OPT_ALLOC_PATH = 10
REMP_OPT_WAIT_SPINS = 11


class RempError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"remp status {status}: {message}")
        self.status = status


def _check(status: int) -> None:
    if status != REMP_OK:
        raise RempError(status, remp_last_error())


def remp_last_error() -> str:
    return _lib.load().remp_last_error().decode()


def _topo_new(T):
    ls = getattr(T, "layer_start", None)
    if ls is None:
        return RempTopo(T.tp, T.pp, None), None
    arr = (C.c_int32 * len(ls))(*ls)
    return RempTopo(T.tp, T.pp, C.cast(arr, C.POINTER(C.c_int32))), arr


_topo_cached = functools.lru_cache(maxsize=512)(_topo_new)


def _topo(T):
    """(remp_topo, keep-alive) for a topology object; marshalled once per distinct (hashable) topology."""
    try:
        return _topo_cached(T)
    except TypeError:
        return _topo_new(T)


def _shape_new(m):
    return RempModelShape(m.num_layers, m.num_kv_heads, m.head_dim, m.block_size, m.elem_bytes)


_shape_cached = functools.lru_cache(maxsize=128)(_shape_new)


def _shape(m):
    try:
        return _shape_cached(m)
    except TypeError:
        return _shape_new(m)


@functools.lru_cache(maxsize=512)
def _caps_cached(caps: tuple):
    return (C.c_int64 * len(caps))(*caps)


def _caps(dst_capacity_blocks):
    return _caps_cached(tuple(int(c) for c in dst_capacity_blocks))


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def remp_shard_bytes(topo, shape, rank: int, num_blocks: int) -> int:
    t, _keep = _topo(topo)
    n = _lib.load().remp_shard_bytes(C.byref(t), C.byref(_shape(shape)), rank, num_blocks)
    if n < 0:
        raise RempError(int(n), remp_last_error())
    return int(n)


def remp_rank_ownership(topo, shape, rank: int):
    """(layer_lo, layer_hi, head_lo, head_hi) of a rank under a topology."""
    t, _keep = _topo(topo)
    out = (C.c_int32 * 4)()
    _check(_lib.load().remp_rank_ownership(C.byref(t), C.byref(_shape(shape)), rank, out))
    return tuple(int(x) for x in out)


def remp_plan_create(src_topo, dst_topo, model_shape, seq_lens, block_tables) -> int:
    """seq_lens int32 [n] and block_tables int32 [n][max_blocks] are CUDA tensors. Returns a plan handle."""
    s, _ks = _topo(src_topo)
    d, _kd = _topo(dst_topo)
    n = int(seq_lens.shape[0])
    maxb = int(block_tables.shape[1]) if block_tables.dim() == 2 else 0
    assert seq_lens.is_cuda and block_tables.is_cuda and seq_lens.is_contiguous() and block_tables.is_contiguous()
    assert str(seq_lens.dtype) == "torch.int32" and str(block_tables.dtype) == "torch.int32"
    bt = RempBlockTables(n, maxb, seq_lens.data_ptr() if n else None, block_tables.data_ptr() if n * maxb else None)
    out = C.c_void_p()
    _check(_lib.load().remp_plan_create(C.byref(s), C.byref(d), C.byref(_shape(model_shape)), C.byref(bt),
                                        C.byref(out)))
    return out.value


def remp_alloc_dst_blocks(plan: int, dst_capacity_blocks: Sequence[int], base_block: int, dst_block_tables,
                          want_total: bool = True, stream=None) -> Optional[int]:
    """dst_block_tables: CUDA int32 tensor shaped like the source tables (written). With want_total the call
    waits for the stream and returns the number of allocated blocks (raising on a device-detected error)."""
    caps = _caps(dst_capacity_blocks)
    total = C.c_int64(-1)
    ptr = dst_block_tables.data_ptr() if dst_block_tables is not None and dst_block_tables.numel() else None
    st = _lib.load().remp_alloc_dst_blocks(plan, caps, base_block, ptr, C.byref(total) if want_total else None,
                                           _stream_ptr(stream))
    _check(st)
    return int(total.value) if want_total else None


def remp_alloc_dst_blocks_preempt(plan: int, dst_capacity_blocks: Sequence[int], base_block: int, dst_block_tables,
                                  preempted, want_counts: bool = True, stream=None):
    """Capacity-constrained allocation: keeps the longest prefix of sequences that fits the smallest pool.
    preempted: CUDA int32 [num_seqs] (written). Returns (total blocks of kept sequences, sequences preempted)
    when want_counts (waits for the stream), else None."""
    caps = _caps(dst_capacity_blocks)
    total, npre = C.c_int64(-1), C.c_int64(-1)
    ptr = dst_block_tables.data_ptr() if dst_block_tables is not None and dst_block_tables.numel() else None
    pre = preempted.data_ptr() if preempted is not None and preempted.numel() else None
    _check(_lib.load().remp_alloc_dst_blocks_preempt(plan, caps, base_block, ptr, pre,
                                                     C.byref(total) if want_counts else None,
                                                     C.byref(npre) if want_counts else None, _stream_ptr(stream)))
    return (int(total.value), int(npre.value)) if want_counts else None


def remp_alloc_dst_blocks_shared(plan: int, dst_capacity_blocks: Sequence[int], base_block: int,
                                 src_num_blocks: int, dst_block_tables, want_total: bool = True, stream=None):
    """Sharing-preserving allocation: entries naming the same source block get the same destination block.
    Returns the number of DISTINCT blocks allocated when want_total (waits for the stream)."""
    caps = _caps(dst_capacity_blocks)
    total = C.c_int64(-1)
    ptr = dst_block_tables.data_ptr() if dst_block_tables is not None and dst_block_tables.numel() else None
    _check(_lib.load().remp_alloc_dst_blocks_shared(plan, caps, base_block, src_num_blocks, ptr,
                                                    C.byref(total) if want_total else None, _stream_ptr(stream)))
    return int(total.value) if want_total else None


def make_shards(buffers, num_blocks: Sequence[int], strides: Optional[Sequence[dict]] = None):
    """Array of remp_shard from CUDA uint8 tensors (one per rank, rank order)."""
    arr = (RempShard * len(buffers))()
    for r, b in enumerate(buffers):
        st = strides[r] if strides else {}
        arr[r] = RempShard(b.data_ptr() if b.numel() else None, int(num_blocks[r]), st.get("layer", 0),
                           st.get("kv", 0), st.get("block", 0), st.get("head", 0), st.get("token", 0))
    return arr


def remp_migrate_kv(plan: int, src_shards, dst_shards, stream=None) -> None:
    """src_shards / dst_shards: arrays from make_shards (rank order). Only enqueues."""
    _check(_lib.load().remp_migrate_kv(plan, src_shards, dst_shards, _stream_ptr(stream)))


def remp_migrate_kv_layers(plan: int, layer_lo: int, layer_hi: int, src_shards, dst_shards, stream=None) -> None:
    """Migrate only layers [layer_lo, layer_hi); each shard describes a buffer holding just the rank's layers
    inside the window (layer-wise streaming). Only enqueues."""
    _check(_lib.load().remp_migrate_kv_layers(plan, layer_lo, layer_hi, src_shards, dst_shards, _stream_ptr(stream)))


def _int32_array(values):
    return (C.c_int32 * len(values))(*[int(v) for v in values])


def remp_plan_partition(plan: int, src_rank_device: Sequence[int], dst_rank_device: Sequence[int], device: int):
    """The plan seen from one device: (recv_items, send_items), int32 arrays of rows
    (src rank, dst rank, layer, head_lo, head_hi, device of the other side)."""
    L = _lib.load()
    sd, dd = _int32_array(src_rank_device), _int32_array(dst_rank_device)
    nr, ns = C.c_int32(), C.c_int32()
    _check(L.remp_plan_partition(plan, sd, dd, device, None, C.byref(nr), None, C.byref(ns)))
    recv = np.zeros((nr.value, 6), dtype=np.int32)
    send = np.zeros((ns.value, 6), dtype=np.int32)
    _check(L.remp_plan_partition(plan, sd, dd, device, recv.ctypes.data, C.byref(nr), send.ctypes.data, C.byref(ns)))
    return recv, send


def remp_migrate_kv_exchange(plan: int, src_rank_device: Sequence[int], dst_rank_device: Sequence[int], device: int,
                             src_shards, dst_shards, stream=None) -> None:
    """remp_migrate_kv for the destination ranks mapped to `device` (the current GPU); sources on other GPUs are
    read in place through addresses this GPU can load from. Only enqueues."""
    _check(_lib.load().remp_migrate_kv_exchange(plan, _int32_array(src_rank_device), _int32_array(dst_rank_device),
                                                device, src_shards, dst_shards, _stream_ptr(stream)))


def remp_plan_status(plan: int, stream=None) -> int:
    return int(_lib.load().remp_plan_status(plan, _stream_ptr(stream)))


def remp_plan_destroy(plan: int) -> None:
    _lib.load().remp_plan_destroy(plan)


def remp_plan_num_items(plan: int) -> int:
    return int(_lib.load().remp_plan_num_items(plan))


def remp_plan_get_items(plan: int) -> np.ndarray:
    n = remp_plan_num_items(plan)
    out = np.zeros((n, 5), dtype=np.int32)
    _check(_lib.load().remp_plan_get_items(plan, out.ctypes.data))
    return out


def remp_plan_traffic(plan: int, total_blocks: int):
    r, w = C.c_int64(), C.c_int64()
    _check(_lib.load().remp_plan_traffic(plan, total_blocks, C.byref(r), C.byref(w)))
    return int(r.value), int(w.value)


def remp_plan_traffic_tokens(plan: int, valid_tokens: int):
    r, w = C.c_int64(), C.c_int64()
    _check(_lib.load().remp_plan_traffic_tokens(plan, valid_tokens, C.byref(r), C.byref(w)))
    return int(r.value), int(w.value)


def remp_plan_set_option(plan: int, key: int, value: int) -> None:
    _check(_lib.load().remp_plan_set_option(plan, key, value))


def remp_release_cached_memory() -> None:
    """Return the library's unused pooled scratch memory to the driver."""
    _check(_lib.load().remp_release_cached_memory())


def remp_kernel_launch_count() -> int:
    return int(_lib.load().remp_kernel_launch_count())


REMP_NOALLOC_MAX_SEQS = 65536


def remp_remap_tables_noalloc(seq_lens, max_blocks_per_seq: int, block_size: int, base_block: int,
                              capacity_blocks: int, dst_block_tables, result, stream=None) -> None:
    """Destination block ids and rewritten tables for callers that cannot allocate device memory (a server
    that gave all HBM to its KV pools, code between decode iterations, a host with a fixed memory budget):
    the scratch is a fixed array inside the library. seq_lens (int32 [n]), dst_block_tables (int32
    [n][max_blocks_per_seq], written) and result (int32 [2]: total, status word, written) are CUDA tensors
    the caller owns. Only enqueues; calls that may overlap on the GPU must be serialised by the caller."""
    n = int(seq_lens.shape[0])
    _check(_lib.load().remp_remap_tables_noalloc(
        seq_lens.data_ptr() if n else None, n, max_blocks_per_seq, block_size, base_block, capacity_blocks,
        dst_block_tables.data_ptr() if dst_block_tables.numel() else None, result.data_ptr(), _stream_ptr(stream)))


REMP_W_REPLICATED, REMP_W_SPLIT_ROWS, REMP_W_SPLIT_COLS, REMP_W_SPLIT_ROW_GROUPS = 0, 1, 2, 3
REMP_W_EVERY_LAYER, REMP_W_FIRST_STAGE, REMP_W_LAST_STAGE = 0, 1, 2


def make_weight_params(params):
    """Array of remp_weight_param from a list of dicts: tensor (host numpy array or CPU torch tensor; [layers][rows]
    [cols] for scope REMP_W_EVERY_LAYER, else [rows][cols]), partition, scope, groups (row groups, for
    REMP_W_SPLIT_ROW_GROUPS)."""
    arr = (RempWeightParam * len(params))()
    for i, p in enumerate(params):
        t = p["tensor"]
        scope = p.get("scope", REMP_W_EVERY_LAYER)
        shape = tuple(t.shape)
        rows, cols = shape[-2], shape[-1]
        e = t.itemsize if isinstance(t, np.ndarray) else t.element_size()
        assert len(shape) == (3 if scope == REMP_W_EVERY_LAYER else 2)
        arr[i] = RempWeightParam(_host_ptr(t), rows * cols * e if scope == REMP_W_EVERY_LAYER else 0, rows, cols, e,
                                 p.get("partition", REMP_W_REPLICATED), p.get("groups", 0), scope)
    return arr


def remp_weight_shard_bytes(topo, num_layers: int, params, rank: int) -> int:
    t, _keep = _topo(topo)
    n = _lib.load().remp_weight_shard_bytes(C.byref(t), num_layers, params, len(params), rank)
    if n < 0:
        raise RempError(int(n), remp_last_error())
    return int(n)


def remp_weight_slice(topo, num_layers: int, params, rank: int, param: int, layer: int = 0):
    """(byte offset in the rank's shard, local rows, local cols) of a parameter (of a layer)."""
    t, _keep = _topo(topo)
    off, rows, cols = C.c_int64(), C.c_int64(), C.c_int64()
    _check(_lib.load().remp_weight_slice(C.byref(t), num_layers, params, len(params), rank, param, layer, C.byref(off),
                                         C.byref(rows), C.byref(cols)))
    return int(off.value), int(rows.value), int(cols.value)


def remp_weights_reshard(topo, num_layers: int, params, dst_shards, stream=None, max_ctas: int = 0) -> int:
    """Materialise every rank's weight shard (CUDA uint8 tensors, one per rank) from the host store described by
    `params` (make_weight_params). Returns the bytes that crossed the host link. Only enqueues when the store is
    page-locked. max_ctas > 0 bounds the gather kernel's grid so that work on other streams runs beside it."""
    t, _keep = _topo(topo)
    ptrs = (C.c_void_p * len(dst_shards))(*[d.data_ptr() if d.numel() else None for d in dst_shards])
    moved = C.c_int64()
    _check(_lib.load().remp_weights_reshard(C.byref(t), num_layers, params, len(params), ptrs, C.byref(moved),
                                            max_ctas, _stream_ptr(stream)))
    return int(moved.value)


def _host_ptr(buf) -> int:
    """Address of a host buffer: a numpy array or a CPU torch tensor (contiguous)."""
    if isinstance(buf, np.ndarray):
        assert buf.flags["C_CONTIGUOUS"]
        return buf.ctypes.data
    assert not buf.is_cuda and buf.is_contiguous()
    return buf.data_ptr()


def remp_reshard_host(src_topo, dst_topo, model_shape, seq_lens, block_tables, src_bufs, src_num_blocks,
                      dst_bufs, dst_num_blocks, base_block: int = 0, window_layers: int = 0):
    """Re-shard a cache held in HOST buffers (numpy arrays or CPU tensors, pinned for full speed), one per
    rank; destination buffers are written in place. Returns (dst_block_tables, total, h2d_bytes, d2h_bytes)."""
    s, _ks = _topo(src_topo)
    d, _kd = _topo(dst_topo)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    n = lens.shape[0]
    maxb = bt.shape[1] if bt.ndim == 2 else 0
    out = np.full((n, maxb), -1, dtype=np.int32)
    ss = (RempHostShard * len(src_bufs))(*[RempHostShard(_host_ptr(b), int(k)) for b, k in zip(src_bufs, src_num_blocks)])
    ds = (RempHostShard * len(dst_bufs))(*[RempHostShard(_host_ptr(b), int(k)) for b, k in zip(dst_bufs, dst_num_blocks)])
    total, up, down = C.c_int64(), C.c_int64(), C.c_int64()
    _check(_lib.load().remp_reshard_host(C.byref(s), C.byref(d), C.byref(_shape(model_shape)), n, maxb,
                                         lens.ctypes.data, bt.ctypes.data, ss, ds, base_block, window_layers,
                                         out.ctypes.data, C.byref(total), C.byref(up), C.byref(down)))
    return out, int(total.value), int(up.value), int(down.value)
