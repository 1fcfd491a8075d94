"""In-tree build of the CUDA library (sm_100a only).

`python -m paper_2609_37062_b200.build` compiles csrc/ into
libdecode_attn.so beside this file with nvcc.  nvcc cross-compiles, so no GPU
is needed to build.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdecode_attn.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    os.makedirs(os.path.join(HERE, "build"), exist_ok=True)
    for src in sources():
        obj = os.path.join(HERE, "build", os.path.basename(src) + ".o")
        cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((src, subprocess.Popen(cmd)))
        objs.append(obj)
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = LIB + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs, "-lcudart"])
    os.replace(tmp, LIB)
    return LIB


TRACE_LIB = os.path.join(HERE, "libdecode_attn_trace.so")


def build_trace() -> str:
    """The same library compiled with -DDA_TRACE: its kernels stamp %globaltimer at a few points of
    every block into a buffer set with decode_attn_trace_set_buffer (see timeline.py).  A diagnostic
    build; the product library carries none of this."""
    if os.path.exists(TRACE_LIB) and all(os.path.getmtime(f) <= os.path.getmtime(TRACE_LIB) for f in _deps()):
        return TRACE_LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = TRACE_LIB + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, *NVCC_FLAGS, "-DDA_TRACE", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
                           *sources(), "-o", tmp, "-lcudart"])
    os.replace(tmp, TRACE_LIB)
    return TRACE_LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
