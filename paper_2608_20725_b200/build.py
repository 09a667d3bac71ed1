"""Builds libim2win.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every .cu under csrc/ is compiled to an object file of its own (in parallel, only when it or a
header changed) and the objects are linked into one shared library.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ_DIR = os.path.join(_HERE, "build")
LIB_PATH = os.path.join(_HERE, "libim2win.so")
HEADER = os.path.join(os.path.dirname(_HERE), "include", "im2win.h")

NVCC_COMPILE_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC",
]
NVCC_LINK_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if not f.endswith(".cu")] + [HEADER]


def _obj_of(src: str) -> str:
    return os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")


def _obj_stale(src: str, obj: str) -> bool:
    if not os.path.exists(obj):
        return True
    t = os.path.getmtime(obj)
    return os.path.getmtime(src) > t or any(os.path.getmtime(h) > t for h in _headers())


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ and link them into one shared library; returns its path."""
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = os.environ.get("IM2WIN_EXTRA_NVCC_FLAGS", "").split()     # e.g. -DIM2WIN_F16_TIMERS
    # objects built with other flags must not be reused; extra flags always mean a rebuild, and so does
    # a library that was last built with extra flags
    stamp = os.path.join(OBJ_DIR, "flags.txt")
    flags_now = " ".join(NVCC_COMPILE_FLAGS + extra)
    flags_old = open(stamp).read() if os.path.exists(stamp) else None
    flags_changed = flags_old is not None and flags_old != flags_now
    if not force and not flags_changed and not extra and not is_stale():
        return LIB_PATH
    os.makedirs(OBJ_DIR, exist_ok=True)
    rebuild_all = force or flags_old != flags_now

    def compile_one(src: str):
        obj = _obj_of(src)
        if not rebuild_all and not _obj_stale(src, obj):
            return 0, ""
        tmp = obj + f".{os.getpid()}.tmp"
        cmd = [nvcc] + NVCC_COMPILE_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", tmp]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if proc.returncode == 0:
            os.replace(tmp, obj)
        return proc.returncode, proc.stdout + proc.stderr

    srcs = sources()
    with ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 4)) as pool:
        results = list(pool.map(compile_one, srcs))
    failed = False
    for rc, out in results:
        if rc != 0 or verbose:
            sys.stderr.write(out)
        failed = failed or rc != 0
    if failed:
        raise RuntimeError("nvcc failed building libim2win.so")
    with open(stamp, "w") as fh:
        fh.write(flags_now)
    tmp = LIB_PATH + f".{os.getpid()}.tmp"
    proc = subprocess.run([nvcc] + NVCC_LINK_FLAGS + [_obj_of(s) for s in srcs] + ["-o", tmp],
                          capture_output=True, text=True)
    if proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
        raise RuntimeError("nvcc failed linking libim2win.so")
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv))
