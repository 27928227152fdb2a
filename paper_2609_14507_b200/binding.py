"""Thin ctypes binding of the C-ABI library (``include/ipkv.h``): argument marshalling only.

Every step of the path runs in the library's CUDA kernels; there is no Python or CPU fallback.
If ``libipkv.so`` is missing or cannot be loaded, :func:`lib` raises.

Tensors are passed as ``torch`` tensors (device or host); this module only takes their
``data_ptr()`` and the current CUDA stream.
"""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libipkv.so")

GQA, MLA = 0, 1
REGION_U, REGION_P, REGION_W = 0, 1, 2
LAYOUT_PLAIN, LAYOUT_TILE = 0, 1
FLAG_NO_HOST_U, FLAG_NO_HOST_P, FLAG_GROW_P = 1, 2, 4
ATTEND_STATIC_SCHEDULE, ATTEND_BALANCE = 1, 2
OK = 0
STATUS_NAMES = {0: "OK", 1: "EINVAL", 2: "ENOMEM", 3: "ERANGE", 4: "ESTATE", 5: "ECUDA", 6: "ETIMEOUT", 7: "EINTERNAL"}

EXPORTS = [
    "ipkv_query_sizes", "ipkv_create", "ipkv_destroy", "ipkv_set_share", "ipkv_reset", "ipkv_append_bulk",
    "ipkv_append", "ipkv_flush", "ipkv_attend_gpu", "ipkv_attend_gpu_sparse", "ipkv_attend_cpu", "ipkv_merge", "ipkv_views", "ipkv_locate", "ipkv_counts",
    "ipkv_read_token", "ipkv_get_stats", "ipkv_profile_enable", "ipkv_profile_read", "ipkv_attend_scratch_bytes", "ipkv_attend_runs", "ipkv_pack_blocks",
    "ipkv_attend_runs_noalloc", "ipkv_noalloc_scratch_limit", "ipkv_roofline_share", "ipkv_roofline_step_time",
    "ipkv_policy_create", "ipkv_policy_destroy", "ipkv_policy_observe", "ipkv_policy_update", "ipkv_policy_prefill_share",
    "ipkv_block_bytes", "ipkv_status_str", "ipkv_last_error", "ipkv_version", "ipkv_probe_read_bandwidth",
    "ipkv_selftest_expire_wait", "ipkv_selftest_fail_next_launch", "ipkv_selftest_declare_bounds", "ipkv_probe_umma",
]


class Config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("kind", C.c_int32), ("n_layers", C.c_int32), ("max_seqs", C.c_int32),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("dim_qk", C.c_int32), ("dim_v", C.c_int32),
        ("block_tokens", C.c_int32), ("window_tokens", C.c_int32), ("chunk_tokens", C.c_int32), ("n_slots", C.c_int32),
        ("max_u_tokens_per_seq", C.c_int64), ("max_p_tokens_per_seq", C.c_int64), ("resident_tokens_per_seq", C.c_int64),
        ("p_initial_tokens_per_seq", C.c_int64),
        ("softmax_scale", C.c_float), ("share_num", C.c_int32), ("share_den", C.c_int32), ("device", C.c_int32),
        ("flags", C.c_uint32),
        ("u_host", C.c_void_p), ("u_bytes", C.c_size_t), ("p_host_pinned", C.c_void_p), ("p_bytes", C.c_size_t),
        ("w_dev", C.c_void_p), ("w_bytes", C.c_size_t), ("resident_dev", C.c_void_p), ("resident_bytes", C.c_size_t),
        ("pp_dev", C.c_void_p), ("pp_bytes", C.c_size_t),
        ("resident_tokens_by_seq", C.POINTER(C.c_int64)),
    ]


class AttendOpts(C.Structure):
    _fields_ = [("kv_splits", C.c_int32), ("flags", C.c_int32), ("side_stream", C.c_void_p),
                ("fold_o_dev", C.c_void_p), ("fold_lse_dev", C.c_void_p), ("append_k_dev", C.c_void_p), ("append_v_dev", C.c_void_p)]


class Extent(C.Structure):
    _fields_ = [("region", C.c_int32), ("layout", C.c_int32), ("first_token", C.c_int64), ("n_tokens", C.c_int64),
                ("region_block", C.c_int64), ("host_ptr", C.c_void_p), ("dev_ptr", C.c_void_p), ("block_bytes", C.c_int64)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "attend_calls", "attend_kernels", "reduce_kernels", "merge_kernels", "append_kernels", "pack_kernels",
        "kv_bytes_attended", "h2d_bytes", "d2h_bytes", "d2d_bytes", "flushes", "flushes_to_u", "fused_appends", "early_launches",
        "p_segments", "p_pinned_bytes", "p_pin_us", "p_grow_waits", "p_grow_wait_us",
        "p_register_us", "p_register_calls", "p_register_max_us")] + [("device_status", C.c_uint32)]


class AttnShape(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("dim_qk", C.c_int32),
                ("dim_v", C.c_int32), ("block_tokens", C.c_int32), ("softmax_scale", C.c_float)]


class Run(C.Structure):
    _fields_ = [("blocks_dev", C.c_void_p), ("n_tokens", C.c_int64)]


class Roofline(C.Structure):
    _fields_ = [("A", C.c_double), ("B", C.c_double), ("C_cpu", C.c_double), ("C_gpu", C.c_double)]


class IpkvError(RuntimeError):
    def __init__(self, status, where, detail=""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".strip())


_lib = None


def lib():
    """Load ``libipkv.so`` (built by ``paper_2609_14507_b200.build``); raises if it is absent.  With IPKV_LIB_VARIANT=checked
    in the environment the bounds-checked build ``libipkv_checked.so`` is loaded instead (same ABI)."""
    global _lib, LIB_PATH
    if _lib is not None:
        return _lib
    if os.environ.get("IPKV_LIB_VARIANT") == "checked":
        LIB_PATH = os.path.join(os.path.dirname(LIB_PATH), "libipkv_checked.so")
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_14507_b200.build` "
                           "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    sig = {
        "ipkv_query_sizes": [C.POINTER(Config), C.POINTER(C.c_size_t)],
        "ipkv_create": [C.POINTER(Config), C.POINTER(vp)],
        "ipkv_destroy": [vp],
        "ipkv_set_share": [vp, i32],
        "ipkv_reset": [vp, i32],
        "ipkv_append_bulk": [vp, i32, i32, vp, vp, i64, i32, i32, vp],
        "ipkv_append": [vp, i32, C.POINTER(i32), i32, vp, vp, vp],
        "ipkv_flush": [vp, i32, i32, vp],
        "ipkv_attend_gpu": [vp, i32, C.POINTER(i32), i32, vp, C.POINTER(AttendOpts), vp, vp, vp],
        "ipkv_attend_gpu_sparse": [vp, i32, C.POINTER(i32), i32, vp, C.POINTER(i64), C.POINTER(i32), i32, C.POINTER(AttendOpts),
                                   vp, vp, vp],
        "ipkv_attend_cpu": [vp, i32, C.POINTER(i32), i32, vp, vp, vp, i32],
        "ipkv_merge": [vp, i32, i32, i32, C.POINTER(vp), C.POINTER(vp), vp, i32, vp, vp],
        "ipkv_views": [vp, i32, i32, C.POINTER(Extent), i32, C.POINTER(i32)],
        "ipkv_locate": [vp, i32, i32, i64, C.POINTER(i32), C.POINTER(i64), C.POINTER(i32)],
        "ipkv_counts": [vp, i32, i32, C.POINTER(i64)],
        "ipkv_read_token": [vp, i32, i32, i64, vp, vp],
        "ipkv_get_stats": [vp, C.POINTER(Stats)],
        "ipkv_selftest_expire_wait": [vp, C.c_uint32, vp],
        "ipkv_selftest_fail_next_launch": [vp],
        "ipkv_selftest_declare_bounds": [vp, i32, i64],
        "ipkv_profile_enable": [vp, i32],
        "ipkv_profile_read": [vp, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(i64)],
        "ipkv_attend_scratch_bytes": [C.POINTER(AttnShape), i32, i32, i64, i32, C.POINTER(C.c_size_t)],
        "ipkv_attend_runs": [C.POINTER(AttnShape), i32, C.POINTER(Run), C.POINTER(i32), vp, i32, vp, C.c_size_t, vp, vp, vp, vp],
        "ipkv_pack_blocks": [C.POINTER(AttnShape), i32, vp, vp, i64, vp, vp],
        "ipkv_attend_runs_noalloc": [C.POINTER(AttnShape), i32, C.POINTER(Run), C.POINTER(i32), vp, i32, vp, vp, vp, vp],
    }
    L.ipkv_version.restype = C.c_char_p
    L.ipkv_version_bytes = lambda: L.ipkv_version()
    for name, args in sig.items():
        f = getattr(L, name)
        f.argtypes = args
        f.restype = C.c_int
    L.ipkv_block_bytes.argtypes = [C.POINTER(AttnShape)]
    L.ipkv_block_bytes.restype = C.c_int64
    L.ipkv_roofline_share.argtypes = [C.POINTER(Roofline), C.c_double]
    L.ipkv_roofline_share.restype = C.c_double
    L.ipkv_roofline_step_time.argtypes = [C.POINTER(Roofline), C.c_double, C.c_double, C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.ipkv_roofline_step_time.restype = C.c_double
    L.ipkv_policy_create.argtypes = [C.POINTER(Roofline), i32, i32, C.POINTER(vp)]
    L.ipkv_policy_destroy.argtypes = [vp]
    L.ipkv_policy_observe.argtypes = [vp, C.c_double, C.c_double]
    L.ipkv_policy_update.argtypes = [vp, C.POINTER(i32), C.POINTER(Roofline)]
    L.ipkv_policy_prefill_share.argtypes = [vp, C.c_double, C.POINTER(i32)]
    for name in ("ipkv_policy_create", "ipkv_policy_destroy", "ipkv_policy_observe", "ipkv_policy_update", "ipkv_policy_prefill_share"):
        getattr(L, name).restype = C.c_int
    L.ipkv_noalloc_scratch_limit.argtypes = []
    L.ipkv_noalloc_scratch_limit.restype = C.c_size_t
    L.ipkv_status_str.argtypes = [C.c_int]
    L.ipkv_status_str.restype = C.c_char_p
    L.ipkv_last_error.argtypes = [vp]
    L.ipkv_last_error.restype = C.c_char_p
    L.ipkv_version.argtypes = []
    L.ipkv_version.restype = C.c_char_p
    _lib = L
    return L


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _ids(seq_ids):
    if isinstance(seq_ids, tuple) and len(seq_ids) == 2 and isinstance(seq_ids[1], int) and not isinstance(seq_ids[0], int):
        return seq_ids                       # already marshalled by seq_id_array()
    arr = (C.c_int32 * len(seq_ids))(*[int(s) for s in seq_ids])
    return arr, len(seq_ids)


def seq_id_array(seq_ids):
    """Marshal a list of sequence ids once; the result can be passed wherever seq_ids is expected."""
    return (C.c_int32 * len(seq_ids))(*[int(s) for s in seq_ids]), len(seq_ids)


def make_config(kind, n_layers, max_seqs, n_q_heads, n_kv_heads, dim_qk, dim_v, *, block_tokens=64,
                window_tokens=256, chunk_tokens=512, n_slots=2, max_u_tokens_per_seq=0, max_p_tokens_per_seq=0,
                resident_tokens_per_seq=0, softmax_scale=0.0, share_num=0, share_den=1, device=0, flags=0,
                p_initial_tokens_per_seq=0, resident_tokens_by_seq=None):
    c = Config()
    c.struct_size = C.sizeof(Config)
    c.kind, c.n_layers, c.max_seqs = kind, n_layers, max_seqs
    c.n_q_heads, c.n_kv_heads, c.dim_qk, c.dim_v = n_q_heads, n_kv_heads, dim_qk, dim_v
    c.block_tokens, c.window_tokens, c.chunk_tokens, c.n_slots = block_tokens, window_tokens, chunk_tokens, n_slots
    c.max_u_tokens_per_seq, c.max_p_tokens_per_seq = max_u_tokens_per_seq, max_p_tokens_per_seq
    c.resident_tokens_per_seq = resident_tokens_per_seq
    c.p_initial_tokens_per_seq = p_initial_tokens_per_seq
    c.softmax_scale = softmax_scale
    c.share_num, c.share_den, c.device, c.flags = share_num, share_den, device, flags
    if resident_tokens_by_seq is not None:                  # per-sequence ring capacities (read by query_sizes / create only)
        if len(resident_tokens_by_seq) != max_seqs:
            raise ValueError("resident_tokens_by_seq needs one entry per sequence")
        c._ring_keepalive = (C.c_int64 * max_seqs)(*[int(x) for x in resident_tokens_by_seq])
        c.resident_tokens_by_seq = C.cast(c._ring_keepalive, C.POINTER(C.c_int64))
    return c


class UmmaTiming(C.Structure):
    _fields_ = [("m", C.c_int32), ("n", C.c_int32), ("n_mma", C.c_int32), ("accumulators", C.c_int32),
                ("issue_cycles", C.c_int64), ("total_cycles", C.c_int64)]


def ipkv_probe_umma(device=0, reps=5):
    """List of dicts: SM clocks for n back-to-back tcgen05.mma of small shapes (see ipkv.h)."""
    out = (UmmaTiming * 64)()
    n = C.c_int32()
    f = lib().ipkv_probe_umma
    f.argtypes = [C.c_int32, C.c_int32, C.POINTER(UmmaTiming), C.c_int32, C.POINTER(C.c_int32)]
    rc = f(device, reps, out, 64, C.byref(n))
    if rc != OK:
        raise IpkvError(rc, "ipkv_probe_umma")
    return [{k: getattr(out[i], k) for k, _ in UmmaTiming._fields_} for i in range(n.value)]


def ipkv_probe_read_bandwidth(device=0, nbytes=1 << 30, reps=10):
    """(best, mean) GB/s of a read-only stream through the attention kernels' copy ring, no arithmetic."""
    best, mean = C.c_double(), C.c_double()
    lib().ipkv_probe_read_bandwidth.argtypes = [C.c_int32, C.c_size_t, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    rc = lib().ipkv_probe_read_bandwidth(device, nbytes, reps, C.byref(best), C.byref(mean))
    if rc != OK:
        raise IpkvError(rc, "ipkv_probe_read_bandwidth")
    return best.value, mean.value


def ipkv_query_sizes(cfg):
    out = (C.c_size_t * 5)()
    rc = lib().ipkv_query_sizes(C.byref(cfg), out)
    if rc != OK:
        raise IpkvError(rc, "ipkv_query_sizes")
    return dict(u=out[0], p=out[1], w=out[2], resident=out[3], pp=out[4])


class Cache:
    """Owner of one ``ipkv_t`` handle; methods carry the C names without the prefix."""

    def __init__(self, cfg):
        self.cfg = cfg
        h = C.c_void_p()
        rc = lib().ipkv_create(C.byref(cfg), C.byref(h))
        if rc != OK:
            raise IpkvError(rc, "ipkv_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().ipkv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def _check(self, rc, where):
        if rc != OK:
            raise IpkvError(rc, where, lib().ipkv_last_error(self._h).decode())

    def set_share(self, num):
        self._check(lib().ipkv_set_share(self._h, num), "ipkv_set_share")

    def reset(self, seq=-1):
        self._check(lib().ipkv_reset(self._h, seq), "ipkv_reset")

    def append_bulk(self, layer, seq, k, v, n_tokens, num0, den0, stream=None):
        self._check(lib().ipkv_append_bulk(self._h, layer, seq, _ptr(k), _ptr(v), n_tokens, num0, den0, _stream(stream)),
                    "ipkv_append_bulk")

    def append(self, layer, seq_ids, k, v, stream=None):
        ids, n = _ids(seq_ids)
        self._check(lib().ipkv_append(self._h, layer, ids, n, _ptr(k), _ptr(v), _stream(stream)), "ipkv_append")

    def flush(self, layer=-1, seq=-1, stream=None):
        self._check(lib().ipkv_flush(self._h, layer, seq, _stream(stream)), "ipkv_flush")

    def attend_gpu(self, layer, seq_ids, q, o_part, lse_part, kv_splits=0, side_stream=None, stream=None,
                   fold_o=None, fold_lse=None, static_schedule=False, force_balance=False, append_k=None, append_v=None):
        """append_k / append_v: one new token per listed sequence, appended first (fused into the kernel where possible)."""
        ids, n = _ids(seq_ids)
        opts = AttendOpts(kv_splits, (ATTEND_STATIC_SCHEDULE if static_schedule else 0) | (ATTEND_BALANCE if force_balance else 0),
                          _stream(side_stream) if side_stream is not None else None, _ptr(fold_o), _ptr(fold_lse),
                          _ptr(append_k), _ptr(append_v))
        self._check(lib().ipkv_attend_gpu(self._h, layer, ids, n, _ptr(q), C.byref(opts), _ptr(o_part), _ptr(lse_part),
                                          _stream(stream)), "ipkv_attend_gpu")

    def attend_gpu_call(self, layer, seq_ids, q, o_part, lse_part, kv_splits=0, side_stream=None, stream=None,
                        fold_o=None, fold_lse=None, static_schedule=False, force_balance=False, append_k=None, append_v=None):
        """The same call as attend_gpu with its arguments marshalled once: returns a function of no arguments that issues
        ipkv_attend_gpu on the given buffers (for loops that call a layer with the same tensors every step)."""
        ids, n = _ids(seq_ids)
        opts = AttendOpts(kv_splits, (ATTEND_STATIC_SCHEDULE if static_schedule else 0) | (ATTEND_BALANCE if force_balance else 0),
                          _stream(side_stream) if side_stream is not None else None, _ptr(fold_o), _ptr(fold_lse),
                          _ptr(append_k), _ptr(append_v))
        fn, check = lib().ipkv_attend_gpu, self._check
        args = (self._h, layer, ids, n, _ptr(q), C.byref(opts), _ptr(o_part), _ptr(lse_part), _stream(stream))
        keep = (opts, ids, q, o_part, lse_part, fold_o, fold_lse, append_k, append_v)      # the buffers stay alive with the call

        def call(_keep=keep):
            rc = fn(*args)
            if rc != OK:
                check(rc, "ipkv_attend_gpu")
        return call

    def attend_gpu_sparse(self, layer, seq_ids, q, blocks_per_row, o_part, lse_part, include_window=True, kv_splits=0,
                          stream=None, fold_o=None, fold_lse=None, static_schedule=False):
        """Attention over the D-window plus the listed whole P blocks of every row (block ordinals in region P)."""
        ids, n = _ids(seq_ids)
        flat, start = [], [0]
        for row in blocks_per_row:
            flat += [int(b) for b in row]
            start.append(len(flat))
        blocks = (C.c_int64 * max(1, len(flat)))(*flat)
        starts = (C.c_int32 * len(start))(*start)
        opts = AttendOpts(kv_splits, ATTEND_STATIC_SCHEDULE if static_schedule else 0, None, _ptr(fold_o), _ptr(fold_lse))
        self._check(lib().ipkv_attend_gpu_sparse(self._h, layer, ids, n, _ptr(q), blocks, starts, 1 if include_window else 0,
                                                 C.byref(opts), _ptr(o_part), _ptr(lse_part), _stream(stream)), "ipkv_attend_gpu_sparse")

    def attend_cpu(self, layer, seq_ids, q_host, o_part_host, lse_part_host, n_threads=0):
        """CPU-side engine over the tokens routed to U; all tensors in host memory."""
        ids, n = _ids(seq_ids)
        self._check(lib().ipkv_attend_cpu(self._h, layer, ids, n, _ptr(q_host), _ptr(o_part_host), _ptr(lse_part_host), n_threads),
                    "ipkv_attend_cpu")

    def merge(self, n_rows, dim_v, o_parts, lse_parts, o_out, lse_out=None, out_is_bf16=False, stream=None):
        ipkv_merge(n_rows, dim_v, o_parts, lse_parts, o_out, lse_out, out_is_bf16, stream, handle=self)

    def views(self, layer, seq):
        n = C.c_int32()
        self._check(lib().ipkv_views(self._h, layer, seq, None, 0, C.byref(n)), "ipkv_views")
        arr = (Extent * max(1, n.value))()
        self._check(lib().ipkv_views(self._h, layer, seq, arr, n.value, C.byref(n)), "ipkv_views")
        return [arr[i] for i in range(n.value)]

    def locate(self, layer, seq, token):
        r, b, o = C.c_int32(), C.c_int64(), C.c_int32()
        self._check(lib().ipkv_locate(self._h, layer, seq, token, C.byref(r), C.byref(b), C.byref(o)), "ipkv_locate")
        return r.value, b.value, o.value

    def counts(self, layer, seq):
        c = (C.c_int64 * 6)()
        self._check(lib().ipkv_counts(self._h, layer, seq, c), "ipkv_counts")
        return dict(n_u=c[0], n_p=c[1], n_w=c[2], n_p_resident=c[3], n_flush=c[4], n_flush_cpu=c[5])

    def read_token(self, layer, seq, token):
        """(K [Hkv][dqk], V [Hkv][dv] or None) of one token as NumPy uint16 bf16 bits."""
        import numpy as np
        cfg = self.cfg
        k = np.zeros((cfg.n_kv_heads, cfg.dim_qk), dtype=np.uint16)
        v = None if cfg.kind == MLA else np.zeros((cfg.n_kv_heads, cfg.dim_v), dtype=np.uint16)
        self._check(lib().ipkv_read_token(self._h, layer, seq, token, k.ctypes.data, v.ctypes.data if v is not None else None),
                    "ipkv_read_token")
        return k, v

    def profile_enable(self, on=True, reduce=False, every=1):
        """Time every `every`-th attention-kernel launch (or, with reduce=True, split-reduce launch) with CUDA events."""
        self._check(lib().ipkv_profile_enable(self._h, ((2 if reduce else 1) + 256 * max(1, int(every))) if on else 0), "ipkv_profile_enable")

    def profile_read(self):
        """(summed attention-kernel milliseconds, launches timed, launches seen) since the last read."""
        ms, nt, nl = C.c_double(), C.c_int64(), C.c_int64()
        self._check(lib().ipkv_profile_read(self._h, C.byref(ms), C.byref(nt), C.byref(nl)), "ipkv_profile_read")
        return ms.value, nt.value, nl.value

    def get_stats(self):
        s = Stats()
        self._check(lib().ipkv_get_stats(self._h, C.byref(s)), "ipkv_get_stats")
        return {n: getattr(s, n) for n, _ in Stats._fields_}

    def selftest_declare_bounds(self, base_id, nbytes):
        self._check(lib().ipkv_selftest_declare_bounds(self._h, base_id, nbytes), "ipkv_selftest_declare_bounds")

    def selftest_fail_next_launch(self):
        self._check(lib().ipkv_selftest_fail_next_launch(self._h), "ipkv_selftest_fail_next_launch")

    def selftest_expire_wait(self, limit_us, stream=None):
        self._check(lib().ipkv_selftest_expire_wait(self._h, limit_us, _stream(stream)), "ipkv_selftest_expire_wait")


def ipkv_merge(n_rows, dim_v, o_parts, lse_parts, o_out, lse_out=None, out_is_bf16=False, stream=None, handle=None):
    n = len(o_parts)
    op = (C.c_void_p * n)(*[_ptr(t) for t in o_parts])
    lp = (C.c_void_p * n)(*[_ptr(t) for t in lse_parts])
    h = handle._h if handle is not None else None
    rc = lib().ipkv_merge(h, n_rows, dim_v, n, op, lp, _ptr(o_out), 1 if out_is_bf16 else 0, _ptr(lse_out), _stream(stream))
    if rc != OK:
        raise IpkvError(rc, "ipkv_merge", lib().ipkv_last_error(h).decode() if h else "")


def ipkv_roofline_share(A, B, C_cpu, C_gpu, L):
    """Eq. 2: the CPU share that balances the two engines at placed length L."""
    return float(lib().ipkv_roofline_share(C.byref(Roofline(A, B, C_cpu, C_gpu)), L))


def ipkv_roofline_step_time(A, B, C_cpu, C_gpu, r, L, t_merge=0.0):
    """Eq. 1: (T, T_CPU, T_GPU) at share r."""
    tc, tg = C.c_double(), C.c_double()
    t = lib().ipkv_roofline_step_time(C.byref(Roofline(A, B, C_cpu, C_gpu)), r, L, t_merge, C.byref(tc), C.byref(tg))
    return float(t), tc.value, tg.value


class Policy:
    """Owner of one ``ipkv_policy_t``: sliding-window feedback on the CPU cost A, marginal share p = B/(A+B)."""

    def __init__(self, A, B, C_cpu, C_gpu, window_steps=256, share_den=64):
        h = C.c_void_p()
        rc = lib().ipkv_policy_create(C.byref(Roofline(A, B, C_cpu, C_gpu)), window_steps, share_den, C.byref(h))
        if rc != OK:
            raise IpkvError(rc, "ipkv_policy_create")
        self._h = h

    def __del__(self):
        if getattr(self, "_h", None):
            lib().ipkv_policy_destroy(self._h)
            self._h = None

    def observe(self, cpu_seconds, cpu_tokens):
        rc = lib().ipkv_policy_observe(self._h, cpu_seconds, cpu_tokens)
        if rc != OK:
            raise IpkvError(rc, "ipkv_policy_observe")

    def update(self):
        """(share numerator, dict of the current model)."""
        num, m = C.c_int32(), Roofline()
        rc = lib().ipkv_policy_update(self._h, C.byref(num), C.byref(m))
        if rc != OK:
            raise IpkvError(rc, "ipkv_policy_update")
        return num.value, dict(A=m.A, B=m.B, C_cpu=m.C_cpu, C_gpu=m.C_gpu)

    def prefill_share(self, L0):
        num = C.c_int32()
        rc = lib().ipkv_policy_prefill_share(self._h, L0, C.byref(num))
        if rc != OK:
            raise IpkvError(rc, "ipkv_policy_prefill_share")
        return num.value


def make_shape(kind, n_q_heads, n_kv_heads, dim_qk, dim_v, block_tokens, softmax_scale=0.0):
    return AttnShape(kind, n_q_heads, n_kv_heads, dim_qk, dim_v, block_tokens, softmax_scale)


def ipkv_block_bytes(shape):
    return int(lib().ipkv_block_bytes(C.byref(shape)))


def ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total_tokens, kv_splits=0):
    out = C.c_size_t()
    rc = lib().ipkv_attend_scratch_bytes(C.byref(shape), n_rows, n_runs, total_tokens, kv_splits, C.byref(out))
    if rc != OK:
        raise IpkvError(rc, "ipkv_attend_scratch_bytes")
    return out.value


def ipkv_attend_runs(shape, runs_per_row, q, scratch, o_part, lse_part, kv_splits=0, status=None, stream=None):
    """runs_per_row: list (one entry per row) of lists of (device pointer or tensor, n_tokens)."""
    flat, start = [], [0]
    for row in runs_per_row:
        for ptr, n in row:
            flat.append(Run(_ptr(ptr), int(n)))
        start.append(len(flat))
    runs = (Run * max(1, len(flat)))(*flat)
    starts = (C.c_int32 * len(start))(*start)
    rc = lib().ipkv_attend_runs(C.byref(shape), len(runs_per_row), runs, starts, _ptr(q), kv_splits, _ptr(scratch),
                                scratch.numel() * scratch.element_size(), _ptr(o_part), _ptr(lse_part), _ptr(status),
                                _stream(stream))
    if rc != OK:
        raise IpkvError(rc, "ipkv_attend_runs")


def _marshal_runs(runs_per_row):
    flat, start = [], [0]
    for row in runs_per_row:
        for ptr, n in row:
            flat.append(Run(_ptr(ptr), int(n)))
        start.append(len(flat))
    return (Run * max(1, len(flat)))(*flat), (C.c_int32 * len(start))(*start)


def ipkv_noalloc_scratch_limit():
    return int(lib().ipkv_noalloc_scratch_limit())


def ipkv_attend_runs_noalloc(shape, runs_per_row, q, o_part, lse_part, kv_splits=0, status=None, stream=None):
    """ipkv_attend_runs for callers that cannot allocate device memory at the call site: same arguments minus the
    scratch buffer, which is a fixed 16 MiB array inside the library (shared by all calls on a device; calls that
    overlap on the GPU race on it).  Raises IpkvError(ERANGE) when the call would need more than that."""
    runs, starts = _marshal_runs(runs_per_row)
    rc = lib().ipkv_attend_runs_noalloc(C.byref(shape), len(runs_per_row), runs, starts, _ptr(q), kv_splits,
                                        _ptr(o_part), _ptr(lse_part), _ptr(status), _stream(stream))
    if rc != OK:
        raise IpkvError(rc, "ipkv_attend_runs_noalloc")


def ipkv_pack_blocks(shape, layout, k, v, n_tokens, dst, stream=None):
    rc = lib().ipkv_pack_blocks(C.byref(shape), layout, _ptr(k), _ptr(v), n_tokens, _ptr(dst), _stream(stream))
    if rc != OK:
        raise IpkvError(rc, "ipkv_pack_blocks")
