"""Builds libsamkv.so (sm_100a only) in-tree with nvcc.  `python -m paper_2508_11661_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libsamkv.so")
DEBUG_LIB_PATH = os.path.join(PKG_DIR, "libsamkv_debug.so")   # same sources with -DSAMKV_DEBUG_CHECKS (test hooks)
SOURCES = ["api.cu", "score.cu", "score_static.cu", "select.cu", "topp.cu", "align.cu", "means.cu", "compact.cu", "attn.cu", "attn_mma.cu", "attn_tc2.cu", "attn_tc3.cu", "attn_tc4.cu"]


def nvcc_path() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "samkv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """debug=True builds libsamkv_debug.so: the same library plus the hooks a test needs to make a bounded wait run out."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not _stale(lib_path):
        return lib_path
    objs = []
    build_dir = os.path.join(PKG_DIR, "build", "debug" if debug else "release")
    os.makedirs(build_dir, exist_ok=True)
    common = [nvcc_path(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if debug:
        common += ["-DSAMKV_DEBUG_CHECKS"]
    if verbose:
        common += ["-Xptxas", "-v"]
    procs = []
    for src in SOURCES:
        obj = os.path.join(build_dir, src.replace(".cu", ".o"))
        objs.append(obj)
        procs.append((src, subprocess.Popen(common + ["-c", os.path.join(CSRC, src), "-o", obj],
                                            stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    subprocess.check_call([nvcc_path(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path] + objs)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, debug=True))
