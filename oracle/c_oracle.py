"""ctypes front-end of the C++ float64 oracle (TEST INFRASTRUCTURE, see ``ipkv_oracle.cpp``).

All bf16 tensors are NumPy ``uint16`` arrays holding the raw bit patterns.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_attend.restype = C.c_int
        L.oracle_attend.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_void_p]
        L.oracle_merge.restype = C.c_int
        L.oracle_merge.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_route_new.restype = C.c_void_p
        L.oracle_route_new.argtypes = [C.c_int64] * 4
        L.oracle_route_free.argtypes = [C.c_void_p]
        L.oracle_route_free.restype = None
        L.oracle_route_set_share.argtypes = [C.c_void_p, C.c_int64]
        L.oracle_route_bulk.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
        L.oracle_route_flush.argtypes = [C.c_void_p]
        L.oracle_route_append.argtypes = [C.c_void_p]
        L.oracle_route_len.argtypes = [C.c_void_p]
        L.oracle_route_len.restype = C.c_int64
        L.oracle_route_counts.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_route_dump.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_threads.argtypes = [C.c_int]
        L.oracle_set_threads.restype = None
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def attend(q, k, v, idx, scale):
    """O1.  q [Hq][dqk], k [n][Hkv][dqk], v [n][Hkv][dv] or None (MLA: V = K[..., :dv] needs dv=...).

    ``v`` may be an int: then V aliases the first ``v`` columns of K (compressed-latent case).
    Returns (O [Hq][dv] float64, LSE [Hq] float64).
    """
    q = _u16(q)
    k = _u16(k)
    Hq, dqk = q.shape
    n, Hkv, dqk2 = k.shape
    assert dqk2 == dqk
    if isinstance(v, (int, np.integer)):
        dv, vptr = int(v), None
    else:
        v = _u16(v)
        assert v.shape[:2] == (n, Hkv)
        dv, vptr = v.shape[2], v.ctypes.data
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    assert idx.ndim == 1 and (idx.size == 0 or (idx.min() >= 0 and idx.max() < n))
    O = np.empty((Hq, dv), dtype=np.float64)
    lse = np.empty((Hq,), dtype=np.float64)
    rc = lib().oracle_attend(q.ctypes.data, k.ctypes.data if n else None, vptr, Hq, Hkv, dqk, dv,
                             idx.ctypes.data if idx.size else None, idx.size, float(scale),
                             O.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_attend rejected its arguments")
    return O, lse


def merge(parts):
    """O2.  parts = [(O_i [rows][dv], lse_i [rows]), ...] -> (O, LSE)."""
    Os = [np.ascontiguousarray(p[0], dtype=np.float64) for p in parts]
    Ls = [np.ascontiguousarray(p[1], dtype=np.float64) for p in parts]
    n_rows, dv = Os[0].shape
    n = len(parts)
    op = (C.c_void_p * n)(*[o.ctypes.data for o in Os])
    lp = (C.c_void_p * n)(*[l.ctypes.data for l in Ls])
    O = np.empty((n_rows, dv), dtype=np.float64)
    lse = np.empty((n_rows,), dtype=np.float64)
    rc = lib().oracle_merge(n_rows, dv, n, op, lp, O.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_merge rejected its arguments")
    return O, lse


REGION_U, REGION_P, REGION_W = 0, 1, 2


class Route:
    """O3.  Routing simulator of one (layer, sequence)."""

    def __init__(self, block, D, num, den):
        self._h = lib().oracle_route_new(block, D, num, den)
        if not self._h:
            raise ValueError("bad routing parameters")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().oracle_route_free(self._h)
            self._h = None

    def set_share(self, num):
        if lib().oracle_route_set_share(self._h, num) != 0:
            raise ValueError("bad share")

    def bulk(self, n0, num0, den0):
        if lib().oracle_route_bulk(self._h, n0, num0, den0) != 0:
            raise ValueError("bulk append rejected")

    def append(self):
        lib().oracle_route_append(self._h)

    def flush(self):
        lib().oracle_route_flush(self._h)

    def __len__(self):
        return int(lib().oracle_route_len(self._h))

    def counts(self):
        c = np.zeros(7, dtype=np.int64)
        lib().oracle_route_counts(self._h, c.ctypes.data)
        return dict(n_u=int(c[0]), n_p=int(c[1]), n_w=int(c[2]), u_blocks=int(c[3]), p_blocks=int(c[4]),
                    n_flush=int(c[5]), n_flush_cpu=int(c[6]))

    def dump(self):
        n = len(self)
        region = np.zeros(n, dtype=np.int8)
        blk = np.zeros(n, dtype=np.int64)
        off = np.zeros(n, dtype=np.int32)
        lib().oracle_route_dump(self._h, region.ctypes.data, blk.ctypes.data, off.ctypes.data)
        return region, blk, off
