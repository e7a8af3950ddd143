"""Builds the CUDA library (sm_100a) in-tree with nvcc.  No GPU is needed to compile."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libkvs.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libkvs_debug.so")   # the same sources with -DKVS_DEBUG (index checks)
SOURCES = ["kvs_api.cu", "kvs_sort.cu", "kvs_build.cu", "kvs_fused.cu", "kvs_refill.cu", "kvs_spec.cu", "kvs_bounds.cu", "kvs_generic.cu", "kvs_sweep.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", _INCLUDE, "-I", _CSRC]


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)] + [os.path.join(_INCLUDE, "kvs.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def _stale_debug() -> bool:
    if not os.path.exists(DEBUG_LIB_PATH):
        return True
    built = os.path.getmtime(DEBUG_LIB_PATH)
    deps = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)] + [os.path.join(_INCLUDE, "kvs.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every kernel for sm_100a and link libkvs.so next to this file (debug: libkvs_debug.so, the
    checked build with -DKVS_DEBUG)."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not (_stale_debug() if debug else _stale()):
        return lib_path
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = os.environ.get("KVS_NVCC_FLAGS", "").split()   # e.g. -DKVS_EVAL_THREADS_CFG=256 when tuning
    if debug:
        extra.append("-DKVS_DEBUG")
    objs, procs = [], []
    for src in SOURCES:
        obj = os.path.join(_HERE, "_build_debug" if debug else "_build", src.replace(".cu", ".o"))
        os.makedirs(os.path.dirname(obj), exist_ok=True)
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(_CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode:
            sys.stderr.write(out)
        failed |= pr.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib_path + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-shared", "-o", tmp, *objs, "-lcudart"])
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
