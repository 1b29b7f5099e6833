"""Build libcomfuse.so (sm_100a only) from csrc/*.cu with nvcc, in-tree.

    python -m paper_2608_03537_b200.build [--force] [--verbose] [--checked]

--checked builds paper_2608_03537_b200/libcomfuse_checked.so (objects under build/obj_checked) with -DCOMFUSE_CHECKED: the
kernels' bounds predicates are compiled in; a predicate that fails records COMFUSE_ERR_BOUNDS in the device status word and
the access is skipped.  COMFUSE_LIB=<path> makes the Python binding load that library instead of libcomfuse.so.

Each translation unit is compiled in parallel to build/obj/*.o and linked into
paper_2608_03537_b200/libcomfuse.so.  A unit is rebuilt when it, or any header in
csrc/ or include/, is newer than its object.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
OBJ_DIR = os.path.join(ROOT, "build", "obj")
LIB_PATH = os.path.join(PKG_DIR, "libcomfuse.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
    "-I", os.path.join(ROOT, "include"),
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if os.path.exists(cand) else "nvcc"


def _newest_header_mtime() -> float:
    m = 0.0
    for d in (CSRC, os.path.join(ROOT, "include")):
        for f in os.listdir(d):
            if f.endswith((".h", ".cuh")):
                m = max(m, os.path.getmtime(os.path.join(d, f)))
    return m


def _compile(src: str, obj: str, verbose: bool, checked: bool = False) -> None:
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", src, "-o", obj]
    if checked:
        cmd.insert(1, "-DCOMFUSE_CHECKED")
    if os.environ.get("COMFUSE_BUILD_TRACE"):   # phase-timestamp tracing build (see fused_params.h: trace)
        cmd.insert(1, "-DCOMFUSE_TRACE")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    obj_dir = OBJ_DIR + "_checked" if checked else OBJ_DIR
    lib_path = os.path.join(PKG_DIR, "libcomfuse_checked.so") if checked else LIB_PATH
    os.makedirs(obj_dir, exist_ok=True)
    sources = sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))
    hdr_m = _newest_header_mtime()
    jobs, objs = [], []
    for f in sources:
        src = os.path.join(CSRC, f)
        obj = os.path.join(obj_dir, f[:-3] + ".o")
        objs.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_m)
        if stale:
            jobs.append((src, obj))
    if jobs:
        with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            list(ex.map(lambda j: _compile(j[0], j[1], verbose, checked), jobs))
    if jobs or not os.path.exists(lib_path):
        cmd = [_nvcc(), "-shared", "-o", lib_path, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
