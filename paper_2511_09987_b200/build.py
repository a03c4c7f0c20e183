"""Compile the CUDA library in-tree with nvcc for sm_100a.

``python -m paper_2511_09987_b200.build`` writes ``paper_2511_09987_b200/libcyc.so``.
nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcyc.so")
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMPILE_FLAGS = [*ARCH_FLAGS, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
LINK_FLAGS = [*ARCH_FLAGS, "-shared", "-Xcompiler", "-fPIC", "--cudart", "static"]
OBJ_DIR = os.path.join(HERE, "_build")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def sources():
    out = []
    for root, _, files in os.walk(CSRC):
        out += [os.path.join(root, f) for f in files if f.endswith((".cu", ".cuh", ".h"))]
    out.append(os.path.join(os.path.dirname(HERE), "include", "cyc.h"))
    return sorted(out)


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(s) > t for s in sources())


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        from concurrent.futures import ThreadPoolExecutor
        cu = [s for s in sources() if s.endswith(".cu")]
        os.makedirs(OBJ_DIR, exist_ok=True)
        nvcc = _nvcc()

        def compile_one(src):  # one translation unit per recurrence, compiled side by side
            obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".%d.o" % os.getpid())
            cmd = [nvcc, *COMPILE_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-c", "-o", obj, src]
            out = subprocess.run(cmd, cwd=HERE, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
            return obj, out

        with ThreadPoolExecutor(max_workers=min(len(cu), os.cpu_count() or 1)) as pool:
            results = list(pool.map(compile_one, cu))
        for obj, out in results:
            if out.stdout and (verbose or out.returncode):
                sys.stderr.write(out.stdout)
            if out.returncode:
                raise subprocess.CalledProcessError(out.returncode, out.args)
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([nvcc, *LINK_FLAGS, "-o", tmp, *[obj for obj, _ in results]], cwd=HERE)
        os.replace(tmp, LIB)
        for obj, _ in results:
            os.remove(obj)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
