"""Builds libzsm.so (sm_100a) in-tree with nvcc.  No GPU is needed to build."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libzsm.so")
OBJ_DIR = os.path.join(HERE, "_build")
SOURCES = ["zsm_api.cu", "zsm_decode.cu", "zsm_decode_split.cu", "zsm_prefill.cu",
           "zsm_prefill_full.cu", "zsm_noalloc.cu", "zsm_fullkv.cu"]
HEADERS = ["zsm_common.cuh", "zsm_decode.cuh", "zsm_decode_split.cuh", "zsm_prefill.cuh",
           "zsm_prefill_full.cuh", "zsm_noalloc.cuh"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC"]


def _obj(src: str) -> str:
    return os.path.join(OBJ_DIR, os.path.splitext(src)[0] + ".o")


def _obj_stale(src: str) -> bool:
    o = _obj(src)
    if not os.path.exists(o):
        return True
    t = os.path.getmtime(o)
    deps = [os.path.join(CSRC, f) for f in [src] + HEADERS]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "zsm.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """One object per source file, compiled side by side and only when older than its source
    or a header; then one link."""
    todo = [f for f in SOURCES if force or _obj_stale(f)]
    if not todo and os.path.exists(LIB) and \
            all(os.path.getmtime(_obj(f)) <= os.path.getmtime(LIB) for f in SOURCES):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    running = []
    for f in todo:
        tmp = _obj(f) + f".tmp{os.getpid()}"
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-c", "-o", tmp, os.path.join(CSRC, f)]
        running.append((f, tmp, subprocess.Popen(cmd)))
    failed = []
    for f, tmp, proc in running:
        if proc.wait() != 0:
            failed.append(f)
        else:
            os.replace(tmp, _obj(f))
    if failed:
        raise RuntimeError("nvcc failed on " + ", ".join(failed))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run([nvcc, "-shared", "-o", tmp] + [_obj(f) for f in SOURCES], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
