"""Builds and loads tests/host_shim.cpp: the product's host-side logic behind a C interface (test-only)."""
import ctypes as C
import os
import subprocess

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "host_shim.cpp")
LIB = os.path.join(HERE, "libhost_shim.so")
_lib = None


def lib():
    global _lib
    if _lib is None:
        deps = [SRC] + [os.path.join(HERE, "..", "paper_2609_14507_b200", "csrc", f) for f in
                        ("plan.hpp", "router.hpp", "layout.cuh", "kernels.h")]
        if not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(d) for d in deps):
            tmp = LIB + ".tmp.%d" % os.getpid()
            subprocess.run(["g++", "-O1", "-std=c++17", "-fPIC", "-shared", "-I/usr/local/cuda/include", "-o", tmp, SRC],
                           check=True)
            os.replace(tmp, LIB)
        L = C.CDLL(LIB)
        L.shim_router_new.restype = C.c_void_p
        L.shim_router_new.argtypes = [C.c_int64] * 4
        for n in ("free", "flush", "append"):
            getattr(L, "shim_router_" + n).argtypes = [C.c_void_p]
            getattr(L, "shim_router_" + n).restype = None
        L.shim_router_set_share.argtypes = [C.c_void_p, C.c_int64]
        L.shim_router_bulk.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
        L.shim_router_len.argtypes = [C.c_void_p]
        L.shim_router_len.restype = C.c_int64
        L.shim_router_counts.argtypes = [C.c_void_p, C.c_void_p]
        L.shim_router_dump.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.shim_plan.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int] + [C.c_void_p] * 8
        L.shim_plan.restype = C.c_int
        L.shim_min_tiles_to_balance.argtypes = [C.c_int64, C.c_int]
        L.shim_min_tiles_to_balance.restype = C.c_int64
        L.shim_tile_chunk_offset.argtypes = [C.c_int32] * 3
        L.shim_tile_chunk_offset.restype = C.c_int64
        L.shim_plain_chunk_offset.argtypes = [C.c_int32] * 3
        L.shim_plain_chunk_offset.restype = C.c_int64
        L.shim_block_bytes.argtypes = [C.c_int32] * 4
        L.shim_block_bytes.restype = C.c_int64
        _lib = L
    return _lib


class Router:
    """The library's router (csrc/router.hpp) with the interface of the oracle's Route."""

    def __init__(self, block, D, num, den):
        self._h = lib().shim_router_new(block, D, num, den)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().shim_router_free(self._h)
            self._h = None

    def set_share(self, num):
        lib().shim_router_set_share(self._h, num)

    def bulk(self, n0, num0, den0):
        lib().shim_router_bulk(self._h, n0, num0, den0)

    def append(self):
        lib().shim_router_append(self._h)

    def flush(self):
        lib().shim_router_flush(self._h)

    def __len__(self):
        return int(lib().shim_router_len(self._h))

    def counts(self):
        c = np.zeros(7, dtype=np.int64)
        lib().shim_router_counts(self._h, c.ctypes.data)
        return dict(n_u=int(c[0]), n_p=int(c[1]), n_w=int(c[2]), u_blocks=int(c[3]), p_blocks=int(c[4]),
                    n_flush=int(c[5]), n_flush_cpu=int(c[6]))

    def dump(self):
        n = len(self)
        region = np.zeros(n, dtype=np.int8); blk = np.zeros(n, dtype=np.int64); off = np.zeros(n, dtype=np.int32)
        lib().shim_router_dump(self._h, region.ctypes.data, blk.ctypes.data, off.ctypes.data)
        return region, blk, off


def plan(rows, n_gh, kv_splits=0, ctas_per_sm=2):
    """rows: list of lists of run token counts -> dict of the planner's tables."""
    row_start = np.zeros(len(rows) + 1, dtype=np.int32)
    segs = []
    for r, row in enumerate(rows):
        segs += list(row)
        row_start[r + 1] = len(segs)
    seg_tokens = np.asarray(segs + [0], dtype=np.int64)
    cap = 1 << 16
    fields = np.zeros((cap, 5), dtype=np.int32)
    cta = np.zeros(148 * ctas_per_sm + 2, dtype=np.int32)
    rg = np.zeros(len(rows) * n_gh + 1, dtype=np.int32)
    seg_out = np.zeros(len(segs) + 1, dtype=np.int32)
    n_segs, n_ctas, table_bytes = C.c_int(), C.c_int(), C.c_int64()
    cta_tiles = np.zeros(148 * ctas_per_sm + 2, dtype=np.int32)
    n = lib().shim_plan(len(rows), row_start.ctypes.data, seg_tokens.ctypes.data, n_gh, kv_splits, ctas_per_sm, cap,
                        fields.ctypes.data, cta.ctypes.data, C.byref(n_ctas), rg.ctypes.data, seg_out.ctypes.data, C.byref(n_segs),
                        cta_tiles.ctypes.data, C.byref(table_bytes))
    assert n >= 0, n
    f = fields[:n]
    return dict(row=f[:, 0], gh=f[:, 1], seg=f[:, 2], tile0=f[:, 3], ntiles=f[:, 4], cta_span_start=cta[:n_ctas.value + 1],
                rg_span_start=rg, seg_tokens=seg_out[:n_segs.value], cta_tiles=cta_tiles[:n_ctas.value],
                table_bytes=table_bytes.value)
