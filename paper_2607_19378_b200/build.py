"""Builds libhyenand.so in-tree with nvcc for sm_100a (no JIT cache involved).

    python -m paper_2607_19378_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libhyenand.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "--use_fast_math", "-Xptxas", "-v"]
# --use_fast_math only affects division/transcendental intrinsics and denormal flushing;
# the transform kernels use neither divisions nor sin/cos on the data path (twiddles come from
# tables computed in double on the host).  Sources that evaluate sines and exponentials of the data
# (kernel synthesis) are compiled without it.
PRECISE = {"synth.cu"}


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _newest_header():
    t = 0.0
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cuh", ".h")):
                t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles and links the library; debug=True builds the checked variant (-DHYENAND_DEBUG) as libhyenand_debug.so."""
    OBJ = os.path.join(HERE, "build_debug" if debug else "build")
    LIB = os.path.join(HERE, "libhyenand_debug.so" if debug else "libhyenand.so")
    os.makedirs(OBJ, exist_ok=True)
    hdr = _newest_header()
    jobs = []
    objs = []
    for src in _sources():
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src[:-3] + ".o")
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            jobs.append((s, o))

    def compile_one(job):
        s, o = job
        flags = [f for f in FLAGS if not (f == "--use_fast_math" and os.path.basename(s) in PRECISE)]
        if debug:
            flags = flags + ["-DHYENAND_DEBUG"]
        r = subprocess.run([NVCC] + flags + ["-c", s, "-o", o], capture_output=True, text=True)
        with open(o[:-2] + ".ptxas.log", "w") as f:
            f.write(r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {s}:\n{r.stderr[-4000:]}")
        if verbose:
            print(r.stderr)
        return o

    if jobs:
        with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            list(ex.map(compile_one, jobs))
    stale = not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs)
    manifest = os.path.join(OBJ, "objects.txt")
    listed = open(manifest).read() if os.path.exists(manifest) else ""
    if jobs or stale or listed != "\n".join(objs):
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs + ["-lcudart", "-ldl"])
        os.replace(tmp, LIB)
        with open(manifest, "w") as f:
            f.write("\n".join(objs))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
