"""In-tree build of libb2blas.so with nvcc for sm_100a (no torch extension machinery: the
library has a plain C ABI and links only the CUDA runtime)."""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")
OBJ_DIR = os.path.join(PKG, "_build")
LIB_PATH = os.path.join(PKG, "libb2blas.so")
DEBUG_LIB_PATH = os.path.join(PKG, "libb2blas_dbg.so")  # the bounds-checking build (-DB2_DEBUG_BOUNDS)

SOURCES = ["api_common.cu", "level1.cu", "gemv.cu", "ger.cu", "tri_f32.cu", "tri_f64.cu", "trsv.cu", "trsv_front.cu", "syr.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _digest() -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    files = sorted(os.listdir(CSRC)) + [os.path.join(INCLUDE, "b2blas.h")]
    for name in files:
        path = name if os.path.isabs(name) else os.path.join(CSRC, name)
        if os.path.isfile(path):
            h.update(name.encode())
            h.update(open(path, "rb").read())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile every .cu under csrc/ and link libb2blas.so; a no-op when sources are unchanged.
    debug_bounds=True builds the bounds-checking variant (libb2blas_dbg.so) instead."""
    lib_path = DEBUG_LIB_PATH if debug_bounds else LIB_PATH
    obj_dir = os.path.join(OBJ_DIR, "dbg") if debug_bounds else OBJ_DIR
    extra = ["-DB2_DEBUG_BOUNDS"] if debug_bounds else []
    stamp = os.path.join(obj_dir, "stamp.txt")
    digest = _digest()
    if not force and os.path.exists(lib_path) and os.path.exists(stamp) and open(stamp).read() == digest:
        return lib_path
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(src):
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{res.stdout}\n{res.stderr}")
        if verbose:
            sys.stderr.write(res.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = lib_path + f".tmp{os.getpid()}"
    res = subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a"],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"link failed:\n{res.stdout}\n{res.stderr}")
    os.replace(tmp, lib_path)
    with open(stamp, "w") as f:
        f.write(digest)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
