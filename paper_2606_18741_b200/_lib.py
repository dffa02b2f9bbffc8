"""Loader of libremp.so (the C-ABI CUDA library). There is no fallback: a missing library is an error."""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libremp.so")

# every symbol include/remp.h declares
EXPORTS = (
    "remp_shard_bytes", "remp_plan_create", "remp_alloc_dst_blocks", "remp_migrate_kv", "remp_plan_status",
    "remp_plan_destroy", "remp_last_error", "remp_plan_num_items", "remp_plan_get_items", "remp_plan_traffic",
    "remp_plan_set_option", "remp_kernel_launch_count", "remp_remap_tables_noalloc", "remp_reshard_host", "remp_migrate_kv_layers", "remp_alloc_dst_blocks_preempt", "remp_alloc_dst_blocks_shared", "remp_plan_traffic_tokens", "remp_release_cached_memory", "remp_rank_ownership", "remp_plan_partition", "remp_migrate_kv_exchange", "remp_weight_shard_bytes", "remp_weight_slice",
    "remp_weights_reshard",
)


class RempTopo(C.Structure):
    _fields_ = [("tp", C.c_int32), ("pp", C.c_int32), ("pp_layer_start", C.POINTER(C.c_int32))]


class RempModelShape(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("block_size", C.c_int32), ("elem_bytes", C.c_int32)]


class RempBlockTables(C.Structure):
    _fields_ = [("num_seqs", C.c_int32), ("max_blocks_per_seq", C.c_int32), ("seq_lens", C.c_void_p),
                ("block_tables", C.c_void_p)]


class RempShard(C.Structure):
    _fields_ = [("base", C.c_void_p), ("num_blocks", C.c_int64), ("stride_layer", C.c_int64),
                ("stride_kv", C.c_int64), ("stride_block", C.c_int64), ("stride_head", C.c_int64),
                ("stride_token", C.c_int64)]


class RempWeightParam(C.Structure):
    _fields_ = [("host_base", C.c_void_p), ("layer_stride", C.c_int64), ("rows", C.c_int64), ("cols", C.c_int64),
                ("elem_bytes", C.c_int32), ("partition", C.c_int32), ("groups", C.c_int32), ("scope", C.c_int32)]


class RempHostShard(C.Structure):
    _fields_ = [("base", C.c_void_p), ("num_blocks", C.c_int64)]


_lib = None


def load():
    """Load the library once; raise if it has not been built (python -m paper_2606_18741_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_18741_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    P = C.POINTER
    L.remp_shard_bytes.argtypes = [P(RempTopo), P(RempModelShape), C.c_int32, C.c_int64]
    L.remp_shard_bytes.restype = C.c_int64
    L.remp_rank_ownership.argtypes = [P(RempTopo), P(RempModelShape), C.c_int32, C.c_void_p]
    L.remp_rank_ownership.restype = C.c_int
    L.remp_plan_create.argtypes = [P(RempTopo), P(RempTopo), P(RempModelShape), P(RempBlockTables), P(C.c_void_p)]
    L.remp_plan_create.restype = C.c_int
    L.remp_alloc_dst_blocks.argtypes = [C.c_void_p, P(C.c_int64), C.c_int32, C.c_void_p, P(C.c_int64), C.c_void_p]
    L.remp_alloc_dst_blocks.restype = C.c_int
    L.remp_alloc_dst_blocks_preempt.argtypes = [C.c_void_p, P(C.c_int64), C.c_int32, C.c_void_p, C.c_void_p,
                                                P(C.c_int64), P(C.c_int64), C.c_void_p]
    L.remp_alloc_dst_blocks_preempt.restype = C.c_int
    L.remp_alloc_dst_blocks_shared.argtypes = [C.c_void_p, P(C.c_int64), C.c_int32, C.c_int64, C.c_void_p,
                                               P(C.c_int64), C.c_void_p]
    L.remp_alloc_dst_blocks_shared.restype = C.c_int
    L.remp_migrate_kv.argtypes = [C.c_void_p, P(RempShard), P(RempShard), C.c_void_p]
    L.remp_migrate_kv.restype = C.c_int
    L.remp_migrate_kv_layers.argtypes = [C.c_void_p, C.c_int32, C.c_int32, P(RempShard), P(RempShard), C.c_void_p]
    L.remp_migrate_kv_layers.restype = C.c_int
    L.remp_plan_partition.argtypes = [C.c_void_p, P(C.c_int32), P(C.c_int32), C.c_int32, C.c_void_p, P(C.c_int32),
                                      C.c_void_p, P(C.c_int32)]
    L.remp_plan_partition.restype = C.c_int
    L.remp_migrate_kv_exchange.argtypes = [C.c_void_p, P(C.c_int32), P(C.c_int32), C.c_int32, P(RempShard), P(RempShard),
                                           C.c_void_p]
    L.remp_migrate_kv_exchange.restype = C.c_int
    L.remp_weight_shard_bytes.argtypes = [P(RempTopo), C.c_int32, P(RempWeightParam), C.c_int32, C.c_int32]
    L.remp_weight_shard_bytes.restype = C.c_int64
    L.remp_weight_slice.argtypes = [P(RempTopo), C.c_int32, P(RempWeightParam), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                    P(C.c_int64), P(C.c_int64), P(C.c_int64)]
    L.remp_weight_slice.restype = C.c_int
    L.remp_weights_reshard.argtypes = [P(RempTopo), C.c_int32, P(RempWeightParam), C.c_int32, P(C.c_void_p), P(C.c_int64),
                                       C.c_int32, C.c_void_p]
    L.remp_weights_reshard.restype = C.c_int
    L.remp_plan_status.argtypes = [C.c_void_p, C.c_void_p]
    L.remp_plan_status.restype = C.c_int
    L.remp_plan_destroy.argtypes = [C.c_void_p]
    L.remp_plan_destroy.restype = None
    L.remp_last_error.argtypes = []
    L.remp_last_error.restype = C.c_char_p
    L.remp_plan_num_items.argtypes = [C.c_void_p]
    L.remp_plan_num_items.restype = C.c_int32
    L.remp_plan_get_items.argtypes = [C.c_void_p, C.c_void_p]
    L.remp_plan_get_items.restype = C.c_int
    L.remp_plan_traffic.argtypes = [C.c_void_p, C.c_int64, P(C.c_int64), P(C.c_int64)]
    L.remp_plan_traffic.restype = C.c_int
    L.remp_plan_traffic_tokens.argtypes = [C.c_void_p, C.c_int64, P(C.c_int64), P(C.c_int64)]
    L.remp_plan_traffic_tokens.restype = C.c_int
    L.remp_plan_set_option.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
    L.remp_plan_set_option.restype = C.c_int
    L.remp_release_cached_memory.argtypes = []
    L.remp_release_cached_memory.restype = C.c_int
    L.remp_kernel_launch_count.argtypes = []
    L.remp_kernel_launch_count.restype = C.c_int64
    L.remp_remap_tables_noalloc.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
    L.remp_remap_tables_noalloc.restype = C.c_int
    L.remp_reshard_host.argtypes = [P(RempTopo), P(RempTopo), P(RempModelShape), C.c_int32, C.c_int32, C.c_void_p,
                                    C.c_void_p, P(RempHostShard), P(RempHostShard), C.c_int32, C.c_int32, C.c_void_p,
                                    P(C.c_int64), P(C.c_int64), P(C.c_int64)]
    L.remp_reshard_host.restype = C.c_int
    _lib = L
    return L
