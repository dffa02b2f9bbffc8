"""Compile the benchmark's measuring aids (tests/native/bench_aid.cu) into libbenchaid.so, linked against
libremp.so. nvcc cross-compiles without a GPU."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
SRC = os.path.join(HERE, "bench_aid.cu")
LIB = os.path.join(HERE, "libbenchaid.so")
PKG = os.path.join(ROOT, "paper_2606_18741_b200")


def build(force: bool = False) -> str:
    from paper_2606_18741_b200 import build as lib_build
    remp_so = lib_build.build()
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(SRC), os.path.getmtime(remp_so)):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler",
           "-fPIC,-Wall,-Wextra", "-shared", "-I", os.path.join(ROOT, "include"), SRC, "-o", LIB + ".tmp",
           "-L", PKG, "-l:libremp.so", "-Xlinker", "-rpath," + PKG, "-lcudart"]
    subprocess.run(cmd, check=True)
    os.replace(LIB + ".tmp", LIB)
    return LIB


class Leg(C.Structure):
    _fields_ = [("src", C.c_void_p), ("dst", C.c_void_p), ("tables", C.c_void_p), ("dst_capacity_blocks", C.c_void_p),
                ("dst_block_tables", C.c_void_p), ("src_shards", C.c_void_p), ("dst_shards", C.c_void_p)]


_lib = None


def load():
    global _lib
    if _lib is None:
        from paper_2606_18741_b200 import _lib as remp_lib
        remp_lib.load()                              # libremp.so first, so the aid binds to the same image
        L = C.CDLL(build())
        L.benchaid_probe_bandwidth.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                               C.c_void_p]
        L.benchaid_probe_bandwidth.restype = C.c_int
        L.benchaid_switch_loop.argtypes = [C.c_void_p, C.POINTER(Leg), C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                           C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.benchaid_switch_loop.restype = C.c_int
        _lib = L
    return _lib


if __name__ == "__main__":
    print(build(force=True))
