"""Builds ``libnm_b200.so`` (the C-ABI library) in-tree with nvcc for sm_100a.

Every ``csrc/*.cu`` is compiled to its own object under ``_build/`` (in parallel, and only when the
source or a header is newer than the object), then the objects are linked into the shared library.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libnm_b200.so")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    deps = glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh"))
    deps.append(os.path.join(os.path.dirname(HERE), "include", "nm.h"))
    return deps


def _obj(src: str, objdir: str = OBJ) -> str:
    return os.path.join(objdir, os.path.splitext(os.path.basename(src))[0] + ".o")


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def build(force: bool = False, verbose: bool = False, defines=(), suffix: str = "") -> str:
    """Compile every .cu under csrc/ into one shared library; returns its path.

    ``defines`` / ``suffix``: extra ``-D`` macros for a second flavour of the library built beside the
    regular one as ``libnm_b200<suffix>.so`` with its own object folder, e.g.
    ``build(defines=("NM_DEBUG_BOUNDS",), suffix="_debug")`` for the self-checking build in which the
    gathering kernels range-check their addresses (load it with ``NM_LIBRARY=<path>``).
    """
    if defines and not suffix:
        raise ValueError("a build with extra macros needs a suffix of its own")
    lib = LIB[:-3] + suffix + ".so"
    objdir = OBJ + suffix
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(objdir, exist_ok=True)
    hdr_t = max(os.path.getmtime(h) for h in _headers())
    flags = ARCH + ["-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"] + [f"-D{d}" for d in defines]
    if verbose:
        flags.append("-Xptxas=-v")

    def compile_one(src):
        obj = _obj(src, objdir)
        if not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_t):
            return
        subprocess.check_call([nvcc] + flags + ["-c", "-o", obj, src])

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        list(pool.map(compile_one, sources()))
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc] + ARCH + ["-shared", "-cudart", "static", "-o", tmp] + [_obj(s, objdir) for s in sources()])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    args = sys.argv[1:]
    defs = tuple(a[2:] for a in args if a.startswith("-D"))
    print(build(force="--force" in args, verbose="-v" in args, defines=defs, suffix="_debug" if defs else ""))
