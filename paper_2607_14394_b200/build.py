"""Builds libdtst.so (sm_100a only) in-tree with nvcc.  `python -m paper_2607_14394_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdtst.so")
SOURCES = ["dtst_api.cu", "dtst_generic.cu", "dtst_fused.cu", "dtst_plane_inst_a.cu", "dtst_plane_inst_b.cu", "dtst_plane_inst_c.cu", "dtst_plane_inst_d.cu", "dtst_row.cu", "dtst_rowg.cu", "dtst_rowl.cu", "dtst_mid.cu", "dtst_midg.cu", "dtst_midmma.cu", "dtst_slab.cu", "dtst_static.cu", "dtst_block.cu", "dtst_block_umma.cu", "dtst_block_mma.cu", "dtst_hostio.cu"]
HEADERS = ["dtst_common.cuh", "dtst_fused.cuh", "dtst_plane.cuh", "dtst_sm100.cuh", "dtst_mma.cuh", os.path.join("..", "..", "include", "dtst.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the DTST library cannot be built")
    return exe


OBJ_DIR = os.path.join(HERE, "build")


def _deps(src: str):
    return [os.path.join(CSRC, src)] + [os.path.join(CSRC, h) for h in HEADERS] + [os.path.abspath(__file__)]


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def needs_build() -> bool:
    return any(_stale(LIB, _deps(s)) for s in SOURCES)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu to an object (in parallel, only the stale ones) and link one shared library next to
    this file; returns its path."""
    if not force and not needs_build():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, os.path.splitext(src)[0] + ".o")
        if not force and not _stale(obj, _deps(src)):
            return obj, ""
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
        return obj, res.stderr

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, SOURCES))
    if verbose:
        for _, log in results:
            if log:
                print(log)
    cmd = [nvcc, "-shared", "-o", LIB] + [obj for obj, _ in results] + ["-lcudart"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


# ---- the plain-C driver (tests/c_driver): proves the library is usable without Python or C++
REPO = os.path.dirname(HERE)
C_DRIVER_SRC = os.path.join(REPO, "tests", "c_driver", "dtst_c_driver.c")
C_DRIVER_BIN = os.path.join(HERE, "dtst_c_driver")


def build_c_driver(force: bool = False) -> str:
    """gcc -std=c99 against include/dtst.h, libdtst.so (found through an $ORIGIN rpath) and the CUDA runtime."""
    build()
    if not force and os.path.exists(C_DRIVER_BIN) and \
            os.path.getmtime(C_DRIVER_BIN) >= max(os.path.getmtime(C_DRIVER_SRC), os.path.getmtime(LIB)):
        return C_DRIVER_BIN
    cuda = os.path.dirname(os.path.dirname(_nvcc()))
    cmd = ["gcc", "-std=c99", "-O2", "-Wall", "-I", os.path.join(REPO, "include"), "-I", os.path.join(cuda, "include"),
           C_DRIVER_SRC, "-o", C_DRIVER_BIN, "-L", HERE, "-ldtst", "-L", os.path.join(cuda, "lib64"), "-lcudart",
           "-Wl,-rpath,$ORIGIN", "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("gcc failed:\n" + res.stdout + res.stderr)
    return C_DRIVER_BIN


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_c_driver(force="--force" in sys.argv))
