"""Build the CUDA library in-tree: paper_2412_01380_b200/libdip.so (sm_100a only).

Each .cu file is compiled to an object of its own (in parallel, and only when it or a header
is newer than the object), then the objects are linked into the shared library.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdip.so")
SOURCES = ["api.cu", "topk.cu", "gemv.cu", "gemv_fused.cu", "gemv_direct_bt.cu", "gemv_int4.cu", "gemv_tc.cu", "gemv_noalloc.cu", "pack.cu", "tier.cu", "rowdot.cu"]
HEADERS = [os.path.join(CSRC, "common.cuh"), os.path.join(CSRC, "gemv_common.cuh"), os.path.join(CSRC, "select_core.cuh"), os.path.join(ROOT, "include", "dip.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def up_to_date() -> bool:
    return not _stale(LIB, [os.path.join(CSRC, s) for s in SOURCES] + HEADERS)


def _compile(src: str, force: bool, verbose: bool) -> str:
    path = os.path.join(CSRC, src)
    obj = os.path.join(OBJ, src[:-3] + ".o")
    if force or _stale(obj, [path] + HEADERS):
        tmp = obj + ".tmp.%d" % os.getpid()
        cmd = [_nvcc(), *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-c", path, "-o", tmp]
        subprocess.run(cmd, check=True)
        os.replace(tmp, obj)
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(lambda s: _compile(s, force, verbose), SOURCES))
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run([_nvcc(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                    *objs, "-o", tmp], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
