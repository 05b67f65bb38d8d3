"""Builds the CUDA library in-tree: paper_2308_13466_b200/libsat_b200.so (sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_NAME = "libsat_b200.so"
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


DEBUG_LIB_NAME = "libsat_b200_dbg.so"   # the same sources with -DSAT_DEBUG_BOUNDS (index checks in the graph kernels)


def lib_path(debug: bool = False) -> str:
    return os.path.join(_HERE, DEBUG_LIB_NAME if debug else LIB_NAME)


def sources():
    return sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")))


def _stale(out: str) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    deps = sources() + glob.glob(os.path.join(_HERE, "csrc", "*.h")) + glob.glob(os.path.join(_HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


LAST_ACTION = None   # "compiled" or "reused": what the most recent build() call did


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles the library when it is older than a source file; debug=True builds the bounds-checking variant."""
    global LAST_ACTION
    out = lib_path(debug)
    if not force and not _stale(out):
        if not debug:
            LAST_ACTION = "reused"
        return out
    if not debug:
        LAST_ACTION = "compiled"
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(_HERE, "build", "dbg" if debug else "rel")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    procs = []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, *(["-DSAT_DEBUG_BOUNDS"] if debug else []), "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for cmd, p in procs:
        log, _ = p.communicate()
        if verbose and log:
            print(log)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd) + "\n" + (log or ""))
    tmp = out + f".tmp{os.getpid()}"
    cmd = [nvcc, "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a", "-ldl"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
