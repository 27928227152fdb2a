"""Build ``libipkv.so`` (the C-ABI library, sm_100a only) in-tree with nvcc.

``python -m paper_2609_14507_b200.build`` compiles every ``csrc/*.cu`` with
``-gencode arch=compute_100a,code=sm_100a -lineinfo`` and links them with the CUDA runtime.
"""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libipkv.so")
LIB_CHECKED = os.path.join(HERE, "libipkv_checked.so")       # the same sources with -DIPKV_CHECKED: bounds-checked kernels
OBJ_DIR = os.path.join(HERE, "build")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _deps_mtime():
    files = glob.glob(os.path.join(CSRC, "*")) + [os.path.join(HERE, "..", "include", "ipkv.h")]
    return max(os.path.getmtime(f) for f in files)


# The CPU engine's tile kernel is compiled once per x86-64 instruction-set level; cpu_engine.cpp picks one at run time.
CPU_KERNEL_LEVELS = (("v4", ["-march=x86-64-v4"]), ("v3", ["-march=x86-64-v3"]), ("base", []))


def cpu_engine_commands(obj_dir):
    """(command, object) pairs that compile the host-only sources (also used by the tests' CPU-engine shim)."""
    out = []
    base = ["g++", "-std=c++17", "-O3", "-fopenmp", "-fPIC", "-Wno-psabi"]
    for src in sorted(glob.glob(os.path.join(CSRC, "*.cpp"))):
        name = os.path.basename(src)[:-4]
        if name == "cpu_engine_amx":
            obj = os.path.join(obj_dir, name + ".o")
            out.append((base + ["-march=x86-64-v4", "-mamx-tile", "-mamx-bf16", "-c", src, "-o", obj], obj))
        elif name == "cpu_engine_kernel":
            for level, flags in CPU_KERNEL_LEVELS:
                obj = os.path.join(obj_dir, f"{name}_{level}.o")
                out.append((base + flags + [f"-DIPKV_CPU_KERNEL=attend_chunk_{level}", "-c", src, "-o", obj], obj))
        else:
            obj = os.path.join(obj_dir, name + ".o")
            out.append((base + ["-c", src, "-o", obj], obj))
    return out


def build(force=False, verbose=False, checked=False):
    """Build libipkv.so, or with checked=True libipkv_checked.so (every kernel compiled with -DIPKV_CHECKED)."""
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    OBJ_DIR = globals()["OBJ_DIR"] + ("_checked" if checked else "")
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _deps_mtime():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    objs = []
    procs = []
    for src in sorted(glob.glob(os.path.join(CSRC, "*.cu"))):
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        cmd = ([NVCC] + FLAGS + (["-DIPKV_CHECKED"] if checked else []) + os.environ.get("IPKV_EXTRA_NVCC", "").split() +
               (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj])
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for cmd, obj in cpu_engine_commands(OBJ_DIR):                       # host-only parts (the CPU-side engine)
        procs.append((cmd[-3], subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run([NVCC, "-shared", "-arch=sm_100a", "-o", tmp] + objs + ["-lcudart", "-lgomp"], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
    print(build(force=True, checked=True))
