"""Compiles csrc/ into libgcnsa.so next to this file (nvcc, sm_100a only).

Every source file is compiled to an object of its own (in parallel, rebuilt only
when it or a header changed) and the objects are linked into the shared
library.  ``build(debug=True)`` makes a second library, libgcnsa_debug.so, with
-DGCNSA_DEBUG: the index-driven kernels then check every gathered column index,
row order entry, row range and scatter position against the bounds they are
given and record the first violation in a status word (gcnsa_debug_status)
instead of making the access.
"""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
LIB = os.path.join(_HERE, "libgcnsa.so")
LIB_DEBUG = os.path.join(_HERE, "libgcnsa_debug.so")
OBJ_DIR = os.path.join(_HERE, "_build")

_ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def sources():
    return sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")) + glob.glob(os.path.join(_HERE, "csrc", "*.cpp")))


def _headers():
    return glob.glob(os.path.join(_HERE, "csrc", "*.h")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def _flags(debug: bool, verbose: bool):
    fl = [*_ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-I" + os.path.join(ROOT, "include")]
    if debug:
        fl.append("-DGCNSA_DEBUG")
    if verbose:
        fl += ["-Xptxas", "-v"]
    return fl


def _object(src: str, debug: bool) -> str:
    return os.path.join(OBJ_DIR, "debug" if debug else "release", os.path.basename(src) + ".o")


def stale(debug: bool = False) -> bool:
    lib = LIB_DEBUG if debug else LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not (force or stale(debug)):
        return lib
    newest_header = max(os.path.getmtime(h) for h in _headers())
    jobs = []
    for src in sources():
        obj = _object(src, debug)
        os.makedirs(os.path.dirname(obj), exist_ok=True)
        if force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header):
            jobs.append(["nvcc", *_flags(debug, verbose), "-c", "-o", obj, src])
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        for rc, cmd in zip(pool.map(lambda c: subprocess.call(c), jobs), jobs):
            if rc != 0:
                raise subprocess.CalledProcessError(rc, cmd)
    subprocess.check_call(["nvcc", *_ARCH, "-shared", "-o", lib, *[_object(s, debug) for s in sources()]])
    return lib
