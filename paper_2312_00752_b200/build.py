"""Compiles the CUDA sources in csrc/ into libssm_scan.so next to this file (sm_100a only, in-tree)."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libssm_scan.so")
# the same library with every tile / global index of the tuned kernels range-checked (-DSSM_DEBUG_BOUNDS)
DEBUG_LIB_PATH = os.path.join(_HERE, "libssm_scan_debug.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-cudart", "static"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), debug_bounds: bool = False) -> str:
    """nvcc -shared of every .cu file; returns the path of the library.  Raises if nvcc fails.  With debug_bounds the
    bounds-checking variant is built into DEBUG_LIB_PATH instead (objects in a directory of their own)."""
    if debug_bounds:
        return _build(DEBUG_LIB_PATH, ".dbg.o", ("-DSSM_DEBUG_BOUNDS", *extra_flags), verbose)
    if not force and not is_stale():
        return LIB_PATH
    return _build(LIB_PATH, ".o", tuple(extra_flags), verbose)


def _build(lib_path: str, obj_suffix: str, extra_flags, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    for src in sources():
        obj = os.path.splitext(src)[0] + obj_suffix
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-I", INCLUDE, "-I", CSRC, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode != 0:
            print(out)
        if pr.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = lib_path + f".tmp{os.getpid()}"
    subprocess.run([nvcc, "-shared", "-cudart", "static", *objs, "-o", tmp], check=True)
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv))
