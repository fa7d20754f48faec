"""Build ``libskv.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every ``csrc/*.cu`` is compiled to an object file of its own (in parallel, rebuilt only when it or a
header is newer) under ``_build/`` and the objects are linked into one shared library."""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ_DIR = os.path.join(_HERE, "_build")
LIB = os.path.join(_HERE, "libskv.so")
LIB_TEST_HOOKS = os.path.join(_HERE, "libskv_testhooks.so")      # the library plus include/skv_test_hooks.h's entry points
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(_HERE, "..", "include", "*.h"))


def _newest_source_mtime() -> float:
    return max(os.path.getmtime(f) for f in sources() + _headers())


def build(force: bool = False, verbose: bool = False, lib: str = LIB, defines=()) -> str:
    """Compile every .cu under csrc/ and link them into one shared library; returns its path.
    ``defines`` (e.g. ``["SKV_TEST_HOOKS"]``) are passed as -D flags and select an object directory of
    their own, so that a differently configured library (``lib``) does not disturb the product's."""
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source_mtime():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("SKV_NVCC_EXTRA", "").split()       # e.g. -DNAME=value for tuning experiments
    extra += [f"-D{d}" for d in defines]
    obj_dir = OBJ_DIR + ("_" + "_".join(sorted(defines)) if defines else "")
    os.makedirs(obj_dir, exist_ok=True)
    hdr_time = max(os.path.getmtime(f) for f in _headers())
    flags_tag = " ".join(NVCC_FLAGS + extra)
    tag_file = os.path.join(obj_dir, "flags.txt")
    same_flags = os.path.exists(tag_file) and open(tag_file).read() == flags_tag

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        fresh = (not force and same_flags and os.path.exists(obj)
                 and os.path.getmtime(obj) >= max(os.path.getmtime(src), hdr_time))
        if not fresh:
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", obj, src]
            subprocess.check_call(cmd)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as pool:
        objs = list(pool.map(compile_one, sources()))
    with open(tag_file, "w") as f:
        f.write(flags_tag)
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs)
    os.replace(tmp, lib)
    return lib


def build_test_hooks(force: bool = False) -> str:
    """The same sources with -DSKV_TEST_HOOKS, as a second library for the test suite."""
    return build(force=force, lib=LIB_TEST_HOOKS, defines=["SKV_TEST_HOOKS"])


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--test-hooks" in sys.argv:
        print(build_test_hooks(force="--force" in sys.argv))
