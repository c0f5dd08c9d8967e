"""In-tree build of ``libmixgcn.so`` for sm_100a with nvcc (cross-compiles without a GPU).

    python -m paper_2501_01951_b200.build [--force] [--verbose] [--debug]

Objects and the shared library are written next to the sources (``csrc/build/`` and
``paper_2501_01951_b200/libmixgcn.so``); both are git-ignored.  ``--debug`` builds the bounds-checked
variant of the same sources instead (``-DMIXGCN_DEBUG_BOUNDS`` -> ``csrc/build_debug/``,
``libmixgcn_debug.so``), which ``MIXGCN_LIBRARY=debug`` makes the binding load.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJDIR = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libmixgcn.so")
OBJDIR_DEBUG = os.path.join(CSRC, "build_debug")
LIB_DEBUG = os.path.join(HERE, "libmixgcn_debug.so")

NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
CFLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC",
          "-I", os.path.relpath(INCLUDE, CSRC), "-I", ".", "--expt-relaxed-constexpr"]   # relative: nvcc runs inside csrc/


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps_mtime():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    return max(os.path.getmtime(h) for h in hs)


def _compile(src, force, verbose, debug=False):
    obj = os.path.join(OBJDIR_DEBUG if debug else OBJDIR, os.path.basename(src)[:-3] + ".o")
    stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), _deps_mtime())
    if stale:
        # compiled from inside csrc/ under its bare file name, so that __FILE__ in error strings is
        # "graph.cu", not a path of the build machine
        cmd = [NVCC, *ARCH, *CFLAGS, *(["-DMIXGCN_DEBUG_BOUNDS"] if debug else []), "-c", os.path.basename(src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        r = subprocess.run(cmd, capture_output=True, text=True, cwd=CSRC)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed on " + src)
    return obj, stale


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    os.makedirs(OBJDIR_DEBUG if debug else OBJDIR, exist_ok=True)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(lambda s: _compile(s, force, verbose, debug), sources()))
    objs = [o for o, _ in results]
    if any(st for _, st in results) or not os.path.exists(lib):
        cmd = [NVCC, *ARCH, "-shared", "-o", lib, *objs]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
