"""Builds libmuloco.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmuloco.so")
LIB_DEBUG = os.path.join(HERE, "libmuloco_debug.so")   # the same sources with -DMULOCO_DEBUG (index checks in the kernels)
SOURCES = ["capi.cu", "elementwise.cu", "outer_sync.cu", "topk.cu", "ns_fp32.cu", "ns_tc.cu", "ns_static.cu"]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: libmuloco cannot be built")
    return cand


def needs_build(lib_path: str = LIB) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "muloco.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, lib_path: str = None, debug: bool = False) -> str:
    """Compile every CUDA source of the package for sm_100a into one shared library.
    debug=True builds libmuloco_debug.so: the same sources with -DMULOCO_DEBUG, i.e. with the
    kernels' index checks compiled in (a failed check raises a status flag, nothing traps)."""
    if lib_path is None:
        lib_path = LIB_DEBUG if debug else LIB
    if not force and lib_path in (LIB, LIB_DEBUG) and not needs_build(lib_path):
        return lib_path
    objs = []
    bdir = os.path.join(HERE, "_build") if lib_path == LIB else (
        os.path.join(HERE, "_build", "debug") if lib_path == LIB_DEBUG else lib_path + ".objs")
    os.makedirs(bdir, exist_ok=True)
    common = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
    if debug:
        common += ["-DMULOCO_DEBUG"]
    if verbose:
        common += ["-Xptxas", "-v"]
    common += os.environ.get("MULOCO_NVCC_FLAGS", "").split()   # extra -D... for tuning studies
    procs = []
    for src in SOURCES:
        obj = os.path.join(bdir, src.replace(".cu", ".o"))
        objs.append(obj)
        procs.append((src, subprocess.Popen(common + ["-c", os.path.join(CSRC, src), "-o", obj],
                                            stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    subprocess.check_call([_nvcc(), "-shared", "-o", lib_path] + objs)
    return lib_path


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
