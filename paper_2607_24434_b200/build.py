"""Builds libdraftexpert.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every translation unit is compiled to an object file of its own (in parallel, skipped when it is newer than every
source and header), then the objects are linked.  ``python -m paper_2607_24434_b200.build [-v] [--checked]``:
``-v`` prints the register / shared-memory report of ptxas, ``--checked`` builds ``libdraftexpert_checked.so``
with ``-DDX_CHECKED`` (explicit bounds checks in the kernels that report through the device status word).
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdraftexpert.so")
LIB_CHECKED = os.path.join(HERE, "libdraftexpert_checked.so")
SOURCES = ["dx_api.cu", "dx_route.cu", "dx_grouped.cu", "dx_wide.cu", "dx_accept.cu", "dx_cache.cu", "dx_controller.cu",
           "dx_eval.cu", "dx_draft_stack.cu", "dx_decode.cu"]


def _headers_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    paths.append(os.path.join(ROOT, "include", "draftexpert.h"))
    paths.append(os.path.abspath(__file__))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    lib = LIB_CHECKED if checked else LIB
    newest = max([_headers_mtime()] + [os.path.getmtime(os.path.join(CSRC, s)) for s in SOURCES])
    if not force and not verbose and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib      # (a library that travelled without its object files is still up to date)
    objdir = os.path.join(HERE, "build", "checked" if checked else "release")
    os.makedirs(objdir, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if checked:
        flags.append("-DDX_CHECKED")
    if verbose:
        flags.append("-Xptxas=-v")
    hdr_t = _headers_mtime()
    jobs = []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(objdir, s[:-3] + ".o")
        stale = force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_t)
        jobs.append((src, obj, stale))

    def compile_one(job):
        src, obj, stale = job
        if not stale:
            return 0, ""
        res = subprocess.run([nvcc, "-c", *flags, "-o", obj, src], capture_output=True, text=True)
        return res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as pool:
        results = list(pool.map(compile_one, jobs))
    failed = False
    for (src, _, _), (rc, log) in zip(jobs, results):
        if log and (verbose or rc != 0):
            sys.stderr.write(f"--- {os.path.basename(src)}\n{log}")
        failed = failed or rc != 0
    if failed:
        raise RuntimeError("nvcc failed building libdraftexpert.so")
    objs = [obj for _, obj, _ in jobs]
    if any(stale for _, _, stale in jobs) or not os.path.exists(lib) or \
            os.path.getmtime(lib) < max(os.path.getmtime(o) for o in objs):
        res = subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib, *objs],
                             capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("linking libdraftexpert.so failed")
    return lib


if __name__ == "__main__":
    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
