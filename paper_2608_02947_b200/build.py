"""Builds libatflash.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2608_02947_b200.build [--force] [--verbose]

Each .cu is compiled to an object file (in parallel) and the objects are linked into
paper_2608_02947_b200/libatflash.so.  The CUDA runtime is linked statically, so the library
loads on a machine without a GPU (its host-only entry points still work there).
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libatflash.so")
SOURCES = ["atf_host.cu", "atf_rope.cu", "atf_decode.cu", "atf_prefill.cu", "atf_prefill_host.cu", "atf_prefill_split.cu", "atf_prefill_pipe.cu"]
HEADERS = [os.path.join(CSRC, "atf_common.cuh"), os.path.join(CSRC, "atf_prefill_pipe.cuh"), os.path.join(ROOT, "include", "atflash.h")]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
EXTRA = os.environ.get("ATF_NVCC_EXTRA", "").split()
FLAGS = EXTRA + ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(src, verbose):
    obj = os.path.join(OBJ, src.replace(".cu", ".o"))
    cmd = [NVCC, *FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    return src, obj, r


def build(force=False, verbose=False):
    os.makedirs(OBJ, exist_ok=True)
    todo = [s for s in SOURCES
            if force or _stale(os.path.join(OBJ, s.replace(".cu", ".o")), [os.path.join(CSRC, s), *HEADERS])]
    if todo:
        with cf.ThreadPoolExecutor(max_workers=len(todo)) as ex:
            for src, obj, r in ex.map(lambda s: _compile(s, verbose), todo):
                if verbose or r.returncode:
                    sys.stderr.write(f"--- {src}\n{r.stdout}{r.stderr}\n")
                if r.returncode:
                    raise RuntimeError(f"nvcc failed on {src}")
    objs = [os.path.join(OBJ, s.replace(".cu", ".o")) for s in SOURCES]
    if force or todo or _stale(LIB, objs):
        cmd = [NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB, *objs]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
