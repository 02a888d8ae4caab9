"""Builds libgsd.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libgsd.so")
LIB_CHECK = os.path.join(PKG, "libgsd_check.so")
OBJ_DIR = os.path.join(PKG, "_build")
SOURCES = ["gsd_api.cu", "gsd_accept.cu", "gsd_accept_sampled.cu", "gsd_draft.cu", "gsd_attn_mma.cu", "gsd_attn_tc.cu", "gsd_attn_plan.cu", "gsd_commit.cu", "gsd_mask.cu", "gsd_unmerge.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the sources that changed and link libgsd.so next to this file.  With `checked`
    the same sources are compiled with -DGSD_BOUNDS_CHECK into libgsd_check.so: the build whose
    kernels check the indices they form and report GSD_DEV_BOUNDS instead of accessing memory
    outside a tensor (used by the tests in place of a memory sanitizer)."""
    obj_dir = OBJ_DIR + ("_check" if checked else "")
    lib = LIB_CHECK if checked else LIB
    extra = ["-DGSD_BOUNDS_CHECK"] if checked else []
    os.makedirs(obj_dir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(ROOT, "include", "gsd.h"))
    jobs, objs = [], []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + headers):
            jobs.append([_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else [])
                        + ["-c", s, "-o", o])

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(run, jobs))
    if force or jobs or _stale(lib, objs):
        tmp = lib + f".tmp{os.getpid()}"
        run([_nvcc(), "-shared", "-o", tmp] + objs
            + ["-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC"])
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
