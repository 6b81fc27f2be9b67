"""Builds the C-ABI CUDA library in-tree: ``python -m paper_2605_21325_b200.build``.

nvcc cross-compiles for sm_100a without a GPU.  The result,
``paper_2605_21325_b200/libtri_inv.so``, is what ``binding`` loads.  Each ``csrc/*.cu`` is compiled to
an object file of its own (in parallel, rebuilt only when it or a header changed) and the objects are
linked into the shared library.

``build(debug=True)`` makes a second library, ``libtri_inv_debug.so``, from the same sources with
``-DTRI_INV_DEBUG``: every shared-memory offset and global store of the kernels is bounds-checked and
mbarrier parities are tracked; a violation raises the device status word (never a trap).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
LIB = os.path.join(PKG, "libtri_inv.so")
LIB_DEBUG = os.path.join(PKG, "libtri_inv_debug.so")
LIB_DEV = os.path.join(PKG, "libtri_inv_dev.so")   # development build with phase clocks (-DTRI_INV_PHASE_CLOCKS)


def sources():
    return sorted(glob.glob(os.path.join(PKG, "csrc", "*.cu")))


def headers():
    return glob.glob(os.path.join(PKG, "csrc", "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(f) > t for f in deps)


def stale(lib: str = LIB) -> bool:
    return _newer(sources() + headers(), lib)


def build(force: bool = False, verbose: bool = False, debug: bool = False, dev: bool = False) -> str:
    lib = LIB_DEV if dev else (LIB_DEBUG if debug else LIB)
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(PKG, "build", "dev" if dev else ("debug" if debug else "release"))
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", os.path.join(PKG, "csrc")]
    flags += os.environ.get("TRI_INV_NVCC_FLAGS", "").split()
    if debug:
        flags.append("-DTRI_INV_DEBUG")
    if dev:
        flags.append("-DTRI_INV_PHASE_CLOCKS")
    if verbose:
        flags += ["-Xptxas", "-v"]
    hdrs = headers()
    jobs = []
    for src in sources():
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        if force or verbose or _newer([src] + hdrs, obj):
            jobs.append([nvcc] + flags + ["-c", src, "-o", obj])

    def run(cmd):
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        return cmd, r.returncode, r.stdout

    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 4))) as ex:
        for cmd, rc, out in ex.map(run, jobs):
            if out.strip() and (verbose or rc != 0):
                sys.stderr.write(out)
            if rc != 0:
                raise subprocess.CalledProcessError(rc, cmd)
    objs = [os.path.join(objdir, os.path.basename(s)[:-3] + ".o") for s in sources()]
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib] + objs)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv, dev="--dev" in sys.argv))
