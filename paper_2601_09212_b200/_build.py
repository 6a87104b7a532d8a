"""Builds libcsd.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC_DIR = os.path.join(_HERE, "csrc")
LIB_DIR = os.path.join(_HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libcsd.so")
SOURCES = [os.path.join(SRC_DIR, "csd_api.cu")]
DEPENDS = SOURCES + [os.path.join(SRC_DIR, "csd_kernels.cuh"), os.path.join(SRC_DIR, "csd_fused.cuh"),
                     os.path.join(SRC_DIR, "csd_tree.cuh"), os.path.join(SRC_DIR, "csd_shard.cuh"),
                     os.path.join(os.path.dirname(_HERE), "include", "csd.h")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared"]


CHECKED_LIB_PATH = os.path.join(LIB_DIR, "libcsd_checked.so")


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(d) > t for d in DEPENDS)


def build_checked_library(force: bool = False) -> str:
    """The same sources with -DCSD_CHECKED: every data-derived index of a logit row is tested before
    the access (see csd_checked_report in csd.h).  For tests; slower than the normal build."""
    return build_library(force=force, path=CHECKED_LIB_PATH, extra=["-DCSD_CHECKED"])


def build_library(force: bool = False, verbose: bool = False, path: str = LIB_PATH, extra=()) -> str:
    """Compiles the library if it is missing or older than its sources.  Safe when several processes
    (one per GPU) start at once: one of them builds, under a file lock, into a temporary file that is
    then moved into place; the others wait and find it fresh."""
    if not (force or is_stale(path)):
        return path
    import fcntl
    os.makedirs(LIB_DIR, exist_ok=True)
    with open(os.path.join(LIB_DIR, ".build.lock"), "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if force or is_stale(path):
                nvcc = os.environ.get("NVCC", "nvcc")
                tmp = f"{path}.{os.getpid()}.tmp"
                cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
                try:
                    subprocess.run(cmd, check=True)
                    os.replace(tmp, path)
                finally:
                    if os.path.exists(tmp):
                        os.remove(tmp)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return path


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
