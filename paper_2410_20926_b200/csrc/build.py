"""Build libta_b200.so (sm_100a only) with nvcc, in-tree next to the package.

Every translation unit is compiled to an object of its own (in parallel, only when it or a
header is newer than the object) under csrc/_build/, then linked into the shared library."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
LIB = os.path.join(os.path.dirname(HERE), "libta_b200.so")
OBJ_DIR = os.path.join(HERE, "_build")
SOURCES = ["ta_api.cu", "ta_simt.cu", "ta_tc.cu", "ta_tc_fused.cu", "ta_tc_pair.cu", "ta_tc_long.cu", "ta_tc_bwd.cu",
           "ta_tc_bwd_long.cu", "ta_simt_bwd.cu", "ta_backward.cu", "ta_noalloc.cu", "ta_selftest.cu", "ta_pad.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", HERE]


def _headers_mtime() -> float:
    deps = [os.path.join(HERE, f) for f in os.listdir(HERE) if f.endswith((".h", ".cuh"))]
    deps.append(os.path.join(ROOT, "include", "ta.h"))
    deps.append(os.path.abspath(__file__))
    return max(os.path.getmtime(d) for d in deps)


def _compile(src: str, force: bool, hdr_t: float, verbose: bool) -> str:
    obj = os.path.join(OBJ_DIR, src[:-3] + ".o")
    path = os.path.join(HERE, src)
    if not force and os.path.exists(obj) and os.path.getmtime(obj) >= max(os.path.getmtime(path), hdr_t):
        return obj
    cmd = ["nvcc"] + (["-Xptxas", "-v"] if verbose else []) + NVCC_FLAGS + ["-c", path, "-o", obj]
    subprocess.run(cmd, check=True)
    return obj


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return _headers_mtime() > t or any(os.path.getmtime(os.path.join(HERE, s)) > t for s in SOURCES)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    hdr_t = _headers_mtime()
    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        objs = list(pool.map(lambda s: _compile(s, force, hdr_t, verbose), SOURCES))
    subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", LIB] + objs, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
