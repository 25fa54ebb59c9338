"""Build libfs_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2502_07021_b200.build [--force] [--debug]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfs_b200.so")
OBJ_DIR = os.path.join(os.path.dirname(HERE), "_build")
SOURCES = ["fs_api.cu", "passes.cu", "batched.cu", "batched_tc.cu", "fused.cu", "fused_log.cu", "resident.cu", "persistent.cu", "shard.cu", "setup.cu", "col_pass_static.cu", "implicit.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _newest_header() -> float:
    roots = [CSRC, os.path.join(os.path.dirname(HERE), "include")]
    t = 0.0
    for root in roots:
        for f in os.listdir(root):
            if f.endswith((".h", ".cuh")):
                t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


DEBUG_LIB = os.path.join(HERE, "libfs_b200_debug.so")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Ordinary library, or with debug=True the checked build (-DFS_DEBUG: canaries behind every owned buffer, launch
    geometry checks, guarded stores) as libfs_b200_debug.so."""
    nvcc = os.environ.get("NVCC", "nvcc")
    obj_dir = os.path.join(OBJ_DIR, "debug") if debug else OBJ_DIR
    lib = DEBUG_LIB if debug else LIB
    flags = NVCC_FLAGS + (["-DFS_DEBUG"] if debug else [])
    os.makedirs(obj_dir, exist_ok=True)
    hdr = _newest_header()
    objs, rebuilt = [], False
    for src in SOURCES:
        sp = os.path.join(CSRC, src)
        op = os.path.join(obj_dir, src.replace(".cu", ".o"))
        objs.append(op)
        if force or not os.path.exists(op) or os.path.getmtime(op) < max(os.path.getmtime(sp), hdr):
            cmd = [nvcc, *flags, "-c", sp, "-o", op]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            subprocess.run(cmd, check=True)
            rebuilt = True
    if rebuilt or not os.path.exists(lib):
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs], check=True)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
