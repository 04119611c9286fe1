"""Compile the CUDA sources into paper_2406_11430_b200/libl2kv.so for sm_100a.

nvcc cross-compiles without a GPU; the CUDA runtime is linked statically so the
library has no dependency beyond the driver.  Every source file is compiled to an
object of its own (in parallel, and only when it or a header changed), then linked.
"""
import glob
import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libl2kv.so")
DEBUG_LIB = os.path.join(HERE, "libl2kv_debug.so")      # the same library with index checks
OBJ_DIR = os.path.join(HERE, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-cudart", "static",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h")) + \
        [os.path.abspath(__file__)]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, out=None, defines=()):
    """out / defines: build a variant (e.g. defines=["L2KV_DEBUG"]) into another file."""
    out = out or LIB
    if not force and not _stale(out, sources() + _headers()):
        return out
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = NVCC_FLAGS + [f"-D{d}" for d in defines] + (["-Xptxas", "-v"] if verbose else [])
    tag = hashlib.sha1(" ".join(flags).encode()).hexdigest()[:10]      # objects of one flag set
    os.makedirs(OBJ_DIR, exist_ok=True)

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, f"{os.path.splitext(os.path.basename(src))[0]}.{tag}.o")
        if force or _stale(obj, [src] + _headers()):
            subprocess.run([nvcc] + flags + ["-c", "-o", obj, src], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    subprocess.run([nvcc] + NVCC_FLAGS + ["-shared", "-o", out] + objs, check=True)
    return out


def build_debug(force=False):
    """The bounds-checked variant: every index check that -DL2KV_DEBUG adds records
    L2KV_ERR_DEBUG_BOUNDS in the workspace and skips the access (nothing traps)."""
    return build(force=force, out=DEBUG_LIB, defines=["L2KV_DEBUG"])


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv))
