"""In-tree build of the CUDA library: nvcc -> paper_2608_11231_b200/liblkv.so (sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "liblkv.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-Xptxas", "-v",
]


def _newer(src: str, dst: str, deps) -> bool:
    if not os.path.exists(dst):
        return True
    t = os.path.getmtime(dst)
    return any(os.path.getmtime(p) > t for p in [src, *deps])


def build(verbose: bool = False, force: bool = False) -> str:
    """Compile every .cu under csrc/ and link liblkv.so; returns the library path."""
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ, exist_ok=True)
    headers = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    objs, procs = [], []
    sources = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    # one stale source means a full rebuild (a few seconds): the library is never a mix of objects from different states
    force = force or any(_newer(src, os.path.join(OBJ, os.path.basename(src)[:-3] + ".o"), headers) for src in sources)
    for src in sources:
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force:
            log = open(obj + ".log", "w")
            procs.append((src, log, subprocess.Popen([nvcc, *NVCC_FLAGS, "-c", src, "-o", obj],
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
    if procs or not os.path.exists(LIB):
        subprocess.run([nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", LIB, *objs], check=True)
    return LIB


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, force="-f" in sys.argv))
