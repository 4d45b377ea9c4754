"""Builds libflashloop.so (sm_100a) in-tree with nvcc.  `python -m paper_2609_29812_b200.build`."""
from __future__ import annotations

import concurrent.futures as cf
import hashlib
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ_DIR = os.path.join(PKG, "build")
LIB_PATH = os.path.join(PKG, "libflashloop.so")
SELFTEST_LIB_PATH = os.path.join(PKG, "libflashloop_selftest.so")
DEBUG_LIB_PATH = os.path.join(PKG, "libflashloop_debug.so")   # the checked build (-DFL_DEBUG_BOUNDS)

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-Xptxas", "-v",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA toolkit is required to build libflashloop.so")
    return exe


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _digest(paths) -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for p in sorted(paths):
        h.update(p.encode())
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ and link the shared library.  Returns its path."""
    srcs = sources()
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    st_dir = os.path.join(CSRC, "selftest")
    headers += [os.path.join(st_dir, f) for f in os.listdir(st_dir)]
    headers.append(os.path.join(ROOT, "include", "flashloop.h"))
    stamp = os.path.join(PKG, "libflashloop.stamp")
    digest = _digest(srcs + headers)
    built = all(os.path.exists(p) for p in (LIB_PATH, DEBUG_LIB_PATH, SELFTEST_LIB_PATH))
    if not force and built and os.path.exists(stamp) and open(stamp).read() == digest:
        return LIB_PATH
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        cmd = [nvcc, *NVCC_FLAGS, "-c", src, "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        with open(obj + ".log", "w") as f:
            f.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with cf.ThreadPoolExecutor(max_workers=min(8, len(srcs))) as ex:
        objs = list(ex.map(compile_one, srcs))
    cmd = [nvcc, "-shared", "-o", LIB_PATH, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    # the checked build: the same objects, with the index validator compiled in
    dbg_obj = os.path.join(OBJ_DIR, "debug_bounds.checked.o")
    r = subprocess.run([nvcc, *NVCC_FLAGS, "-DFL_DEBUG_BOUNDS", "-c", os.path.join(CSRC, "debug_bounds.cu"), "-o", dbg_obj],
                       capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on the checked build of debug_bounds.cu:\n{r.stdout}\n{r.stderr}")
    dbg_objs = [dbg_obj if os.path.basename(o) == "debug_bounds.o" else o for o in objs]
    r = subprocess.run([nvcc, "-shared", "-o", DEBUG_LIB_PATH, *dbg_objs, "-gencode", "arch=compute_100a,code=sm_100a"],
                       capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link of the checked build failed:\n{r.stdout}\n{r.stderr}")
    # tensor-path self-test kernels: a library of their own, loaded only by a GPU test
    st_dir = os.path.join(CSRC, "selftest")
    st_srcs = sorted(os.path.join(st_dir, f) for f in os.listdir(st_dir) if f.endswith(".cu"))
    cmd = [nvcc, *NVCC_FLAGS, "-shared", "-o", SELFTEST_LIB_PATH, *st_srcs]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"self-test library failed to build:\n{r.stdout}\n{r.stderr}")
    with open(stamp, "w") as f:
        f.write(digest)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
