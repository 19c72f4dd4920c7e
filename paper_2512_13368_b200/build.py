"""Builds the CUDA library in-tree: ``paper_2512_13368_b200/libblossom.so`` (sm_100a only).

Run as ``python -m paper_2512_13368_b200.build`` or call ``build()``; nvcc cross-compiles
without a GPU.  The shared object is loaded with ctypes (see ``binding.py``).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libblossom.so")
OBJ = os.path.join(HERE, "_build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]
# --use_fast_math only affects the fp32 attention kernels' exp2f/logf/division; the fp64 block
# scoring is untouched by it.


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    headers = glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(HERE, "..", "include", "blossom.h")]
    objs = []
    procs = []
    live = {os.path.basename(x)[:-3] + ".o" for x in sources()}
    for f in os.listdir(OBJ):  # stale objects of sources that no longer exist
        if f.endswith(".o") and f not in live:
            os.remove(os.path.join(OBJ, f))
    for src in sources():
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            log = open(obj + ".log", "w")
            procs.append((src, log, subprocess.Popen([nvcc] + NVCC_FLAGS + ["-c", src, "-o", obj],
                                                     stdout=log, stderr=subprocess.STDOUT)))
    failed = False
    for src, log, p in procs:
        rc = p.wait()
        log.close()
        text = open(log.name).read()
        if rc != 0:
            failed = True
            sys.stderr.write(text)
        elif verbose:
            sys.stdout.write(text)
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _stale(LIB, objs):
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs + ["-cudart", "static"])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
