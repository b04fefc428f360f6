"""In-tree build of the C-ABI CUDA library (libtca.so) for sm_100a with nvcc.

``python -m paper_2512_09238_b200._build`` (or :func:`build`) compiles every ``csrc/*.cu``
into an object file next to a stamp of its inputs and links them into
``paper_2512_09238_b200/libtca.so``.  Objects are rebuilt only when a source or header
changed.  nvcc cross-compiles, so this works on a machine without a GPU.

``build(debug_bounds=True)`` (``--debug-bounds`` on the command line) builds the range-checked
variant ``libtca_dbg.so`` from the same sources with ``-DTCA_DEBUG_BOUNDS``: every index and
offset a kernel reads from memory is compared with its range before use (see include/tca.h).
"""
from __future__ import annotations

import concurrent.futures as cf
import hashlib
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")
BUILD = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libtca.so")
LIB_DEBUG = os.path.join(PKG, "libtca_dbg.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC",
    "-I", INCLUDE, "-I", CSRC, "-DTCA_BUILD",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _digest(paths) -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for p in sorted(paths):
        with open(p, "rb") as f:
            h.update(p.encode())
            h.update(f.read())
    return h.hexdigest()


def _compile(src: str, headers, verbose: bool, extra, build_dir: str = BUILD) -> str:
    obj = os.path.join(build_dir, os.path.basename(src)[:-3] + ".o")
    stamp = obj + ".stamp"
    want = _digest([src, *headers]) + " ".join(extra)
    if os.path.exists(obj) and os.path.exists(stamp) and open(stamp).read() == want:
        return obj
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", src, "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}")
    with open(stamp, "w") as f:
        f.write(want)
    return obj


def build(verbose: bool = False, ptxas_info: bool = False, debug_bounds: bool = False) -> str:
    """Compile and link libtca.so (or, with debug_bounds, libtca_dbg.so); returns its path."""
    build_dir = BUILD + "_dbg" if debug_bounds else BUILD
    lib = LIB_DEBUG if debug_bounds else LIB
    os.makedirs(build_dir, exist_ok=True)
    srcs = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    extra = ["-Xptxas", "-v"] if ptxas_info else []
    if debug_bounds:
        extra.append("-DTCA_DEBUG_BOUNDS")
    with cf.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(lambda s: _compile(s, headers, verbose or ptxas_info, extra, build_dir), srcs))
    newest = max(os.path.getmtime(o) for o in objs)
    if not os.path.exists(lib) or os.path.getmtime(lib) < newest:
        cmd = [_nvcc(), "-shared", "-o", lib, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
               "-Xcompiler", "-fPIC", "-lcuda"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError(f"link of {os.path.basename(lib)} failed")
    return lib


if __name__ == "__main__":
    print(build(verbose=True, ptxas_info="--ptxas" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
