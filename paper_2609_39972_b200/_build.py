"""Builds ``libubt.so`` in-tree with nvcc for sm_100a (no JIT cache, no torch extension machinery)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libubt.so")
CHECKED_LIB = os.path.join(HERE, "libubt_checked.so")   # -DUBT_BOUNDS_CHECK debug build
SOURCES = ["ubt_api.cu", "ubt_topk.cu", "ubt_tree.cu", "ubt_verify.cu", "ubt_verify_path.cu", "ubt_noalloc.cu",
           "ubt_selector.cu", "ubt_lmhead.cu"]
HEADERS = ["ubt_common.cuh", "ubt_internal.h", "ubt_merge.cuh", "ubt_ring.cuh", "ubt_pick.cuh", "ubt_tc.cuh", os.path.join("..", "..", "include", "ubt.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every kernel for sm_100a and link the shared library; returns its path.

    ``checked=True`` builds ``libubt_checked.so`` with range-checked array views (a debugging aid).
    """
    target = CHECKED_LIB if checked else LIB
    if not checked and not force and not is_stale():
        return LIB
    objs = []
    procs = []
    for s in SOURCES:
        obj = os.path.join(CSRC, s.replace(".cu", ".chk.o" if checked else ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, *(["-DUBT_BOUNDS_CHECK"] if checked else []), "-c", os.path.join(CSRC, s),
               "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for s, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(out)
        failed = failed or p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed building libubt")
    tmp = target + f".{os.getpid()}.tmp"
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
                           "-lcudart"])
    os.replace(tmp, target)
    return target


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
