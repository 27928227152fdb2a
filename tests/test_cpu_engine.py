"""The CPU-side in-place attention engine (Sec. 6.1) against the oracle, on the host alone: grouped-query and
compressed-latent shapes, several runs with ragged ends, token counts around the engine's tile and chunk sizes."""
import ctypes as C
import os
import subprocess

import numpy as np
import pytest

from oracle import c_oracle
from paper_2609_14507_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "..", "paper_2609_14507_b200", "csrc")
LIB = os.path.join(HERE, "libcpu_engine_shim.so")


def _lib():
    from paper_2609_14507_b200 import build as lib_build
    obj_dir = os.path.join(HERE, "..", "paper_2609_14507_b200", "build")
    os.makedirs(obj_dir, exist_ok=True)
    cmds = lib_build.cpu_engine_commands(obj_dir)
    deps = [os.path.join(HERE, "cpu_engine_shim.cpp"), os.path.join(CSRC, "cpu_engine.h"), os.path.join(CSRC, "cpu_engine.cpp"),
            os.path.join(CSRC, "cpu_engine_kernel.cpp"), os.path.join(CSRC, "cpu_engine_amx.cpp")]
    if not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(d) for d in deps):
        for cmd, _ in cmds:
            subprocess.run(cmd, check=True)
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", tmp, os.path.join(HERE, "cpu_engine_shim.cpp")] +
                       [obj for _, obj in cmds], check=True)
        os.replace(tmp, LIB)
    return C.CDLL(LIB)


def run_engine(sh, k, v, q, runs, bt, threads=0, reps=1, seconds=None):
    L = _lib()
    n = k.shape[0]
    o = np.zeros((sh.n_q_heads, sh.dim_v), np.float32)
    lse = np.zeros(sh.n_q_heads, np.float32)
    rt = np.asarray(runs, np.int64)
    best = C.c_double()
    rc = L.shim_cpu_attend(sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v, bt, C.c_float(np.float32(sh.scale)), C.c_int64(n),
                           k.ctypes.data_as(C.c_void_p), None if v is None else v.ctypes.data_as(C.c_void_p), len(runs),
                           rt.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), o.ctypes.data_as(C.c_void_p),
                           lse.ctypes.data_as(C.c_void_p), threads, reps, C.byref(best))
    assert rc == 0, rc
    if seconds is not None:
        seconds.append(best.value)
    return o, lse


@pytest.mark.parametrize("shape,bt,runs", [
    (synth.Shape("g8", "gqa", 1, 16, 2, 128, 128, 128 ** -0.5), 64, [1000]),
    (synth.Shape("g4", "gqa", 1, 8, 2, 128, 128, 128 ** -0.5), 16, [17, 1, 300, 2049]),
    (synth.Shape("g1", "gqa", 1, 4, 4, 64, 64, 64 ** -0.5), 32, [33, 4096 + 5]),
    (synth.Shape("g16", "gqa", 1, 32, 2, 128, 128, 128 ** -0.5), 64, [15, 16, 31]),
    (synth.Shape("mla", "mla", 1, 16, 1, 576, 512, 192 ** -0.5), 64, [700, 129]),
    (synth.Shape("mla5", "mla", 1, 5, 1, 576, 512, 192 ** -0.5), 16, [2100]),
])
def test_cpu_engine_matches_oracle(shape, bt, runs):
    n = sum(runs)
    k, v = synth.host_kv(shape, n, seed=31 + n)
    q = synth.host_q(shape, 1, seed=32 + n)[0]
    o, lse = run_engine(shape, k, v, q, runs, bt)
    scale = float(np.float32(shape.scale))
    o_ref, l_ref = c_oracle.attend(q, k, shape.dim_v if v is None else v, np.arange(n), scale)
    assert np.abs(o - o_ref).max() < 2e-5 and np.abs(lse - l_ref).max() < 2e-5


def test_cpu_engine_extremes():
    sh = synth.Shape("g8", "gqa", 1, 8, 1, 128, 128, 128 ** -0.5)
    k, v = synth.host_kv(sh, 300, seed=5)
    q = synth.host_q(sh, 1, seed=6)[0]
    # one token; an empty set; thread counts
    o, lse = run_engine(sh, k[:1], v[:1], q, [1], 64)
    o_ref, l_ref = c_oracle.attend(q, k[:1], v[:1], np.arange(1), float(np.float32(sh.scale)))
    assert np.abs(o - o_ref).max() < 1e-6 and np.abs(lse - l_ref).max() < 1e-5
    o, lse = run_engine(sh, k[:0], v[:0], q, [], 64)
    assert np.all(o == 0) and np.all(np.isneginf(lse))
    a = run_engine(sh, k, v, q, [300], 64, threads=1)
    b = run_engine(sh, k, v, q, [300], 64, threads=4)
    np.testing.assert_array_equal(a[0], b[0])
    # a dominant key: the weights collapse onto one token, large scores must not overflow
    kb = k.copy(); kb[123] = synth.normal_bf16(np.random.default_rng(1), (1, 128)) * 0 + np.uint16(0x4120)     # 10.0 everywhere
    qb = np.full_like(q, np.uint16(0x4120))
    o, lse = run_engine(sh, kb, v, qb, [300], 64)
    o_ref, l_ref = c_oracle.attend(qb, kb, v, np.arange(300), float(np.float32(sh.scale)))
    assert np.abs(o - o_ref).max() < 1e-4 and np.abs(lse - l_ref).max() / abs(l_ref).max() < 1e-6


@pytest.mark.parametrize("level", ["v4", "v3", "base"])
def test_every_kernel_level_matches_the_oracle(level):
    """The engine picks the best tile kernel the host has (the AMX one where there is a tile unit), so on such a host the
    vector kernels would go untested: the same parity cases run once more with each level forced (IPKV_CPU_KERNEL, read
    when the engine is first used: a child process).  A level the host cannot run falls back to the host's best."""
    import sys
    _lib()          # built once, here, not by the children at the same time
    root = os.path.dirname(HERE)
    env = dict(os.environ, IPKV_CPU_KERNEL=level)
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", os.path.join(HERE, "test_cpu_engine.py"), "-k",
                        "matches_oracle or extremes or ragged_steps" ], env=env, cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]


@pytest.mark.parametrize("shape,bt,runs", [
    (synth.Shape("g8", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5), 64, [64, 31, 33, 1, 95, 2048 + 7]),     # steps straddle blocks and runs
    (synth.Shape("g2d64", "gqa", 1, 4, 2, 64, 64, 64 ** -0.5), 32, [32, 32, 5, 64]),
    (synth.Shape("g16", "gqa", 1, 16, 1, 128, 128, 128 ** -0.5), 128, [4096 + 40]),                     # several items of 2048 tokens
    (synth.Shape("mla16", "mla", 1, 16, 1, 576, 512, 192 ** -0.5), 32, [31, 2049]),
    (synth.Shape("g32", "gqa", 1, 32, 1, 128, 128, 128 ** -0.5), 64, [200]),                            # more heads than one tile holds: done in slices of 16
])
def test_cpu_engine_ragged_steps_and_wide_groups(shape, bt, runs):
    """Shapes around the 32-token steps of the tile-unit kernel: runs that end inside a step, blocks smaller than a step,
    steps that straddle a block boundary, groups that fill all 16 tile rows, and a group wider than that."""
    n = sum(runs)
    k, v = synth.host_kv(shape, n, seed=77 + n)
    q = synth.host_q(shape, 1, seed=78 + n)[0]
    o, lse = run_engine(shape, k, v, q, runs, bt)
    o_ref, l_ref = c_oracle.attend(q, k, shape.dim_v if v is None else v, np.arange(n), float(np.float32(shape.scale)))
    assert np.abs(o - o_ref).max() < 2e-5 and np.abs(lse - l_ref).max() < 2e-5
