"""In-tree build of libs4c.so (hand-written CUDA for sm_100a) with nvcc.  No JIT cache, no torch types."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INC = os.path.join(os.path.dirname(_HERE), "include")
_LIB = os.path.join(_HERE, "libs4c.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math", "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall"]


def lib_path() -> str:
    return _LIB


def sources():
    return sorted(glob.glob(os.path.join(_CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(_CSRC, "*.cuh")) + glob.glob(os.path.join(_CSRC, "*.h")) + \
        glob.glob(os.path.join(_INC, "*.h"))


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ for sm_100a and link libs4c.so next to this file."""
    deps = _deps()
    if not sources():
        raise RuntimeError("no CUDA sources found under " + _CSRC)
    newest = max(os.path.getmtime(p) for p in deps)
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= newest:
        return _LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    for src in sources():
        obj = os.path.splitext(src)[0] + ".o"
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, "-I", _INC, "-I", _CSRC, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd)))
    for src, p in procs:
        if p.wait() != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-lcudart"], check=True)
    os.replace(tmp, _LIB)
    return _LIB
