"""In-tree build of libdynakv.so for sm_100a with nvcc (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libdynakv.so")
OBJ = os.path.join(_HERE, "_build")
SOURCES = ["api.cu", "build_kernels.cu", "decode_kernels.cu", "split_kernel.cu", "assign_tc.cu", "attn_kernels.cu", "front_kernels.cu", "noalloc_attend.cu", "tier.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    tt = os.path.getmtime(target)
    return any(os.path.getmtime(d) > tt for d in deps)


LIB_CHECKED = os.path.join(_HERE, "libdynakv_checked.so")
OBJ_CHECKED = os.path.join(_HERE, "_build_checked")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Build libdynakv.so, or with checked=True libdynakv_checked.so: the same sources with -DDYNAKV_CHECKED (every
    table-derived index tested before use), which the test suite runs a few cases against."""
    LIB, OBJ = (LIB_CHECKED, OBJ_CHECKED) if checked else (globals()["LIB"], globals()["OBJ"])
    flags = NVCC_FLAGS + (["-DDYNAKV_CHECKED"] if checked else [])
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(os.path.dirname(_HERE), "include", "dynakv.h"))
    srcs = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    objs = []
    jobs = []
    for s in srcs:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ, s.replace(".cu", ".o"))
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        r = subprocess.run(["nvcc", *flags, "-c", src, "-o", obj], capture_output=True, text=True)
        log = r.stdout + r.stderr
        with open(obj + ".log", "w") as f:
            f.write(log)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{log}")
        if verbose:
            print(log)
        return obj

    if jobs:
        with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            list(ex.map(compile_one, jobs))
    if jobs or _stale(LIB, objs):
        subprocess.check_call(["nvcc", "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
                               "-lcudart"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
