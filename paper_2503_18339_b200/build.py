"""In-tree build of the GranQ CUDA library for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libgranq.so")
OBJ_DIR = os.path.join(HERE, "_build")
SOURCES = ["granq_api.cu", "granq_flat.cu", "granq_staged.cu", "granq_l2wave.cu", "granq_colwalk.cu",
           "granq_cluster.cu", "granq_accumulate.cu", "granq_rows.cu", "granq_weights.cu", "granq_selftest.cu", "granq_noalloc.cu"]
HEADERS = ["granq_device.cuh", "granq_internal.h"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC"]


def _deps():
    return [os.path.join(CSRC, f) for f in HEADERS] + [os.path.join(INCLUDE, "granq.h")]


def _newer(path: str, than: float) -> bool:
    return os.path.getmtime(path) > than


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(_newer(d, t) for d in [os.path.join(CSRC, f) for f in SOURCES] + _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu (one object per source, in parallel) and link libgranq.so beside this file;
    returns its path.  Objects are kept in _build/ and reused while their source and the headers are older."""
    if not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        path = os.path.join(CSRC, src)
        if not force and not verbose and os.path.exists(obj):
            t = os.path.getmtime(obj)
            if not any(_newer(d, t) for d in [path] + _deps()):
                return obj
        cmd = [nvcc, *NVCC_FLAGS, "-I", INCLUDE, "-c", path, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.check_call(cmd)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-o", tmp] + objs)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
