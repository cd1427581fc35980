"""Builds the CUDA library in-tree: nvcc for sm_100a -> paper_2507_07149_b200/libdaf.so."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libdaf.so")
HEADERS = [os.path.join(CSRC, h) for h in ("common.cuh", "compress_shared.cuh", "compress_stream.cuh", "compress_general.cuh", "compress_twopass.cuh", "compress_twowidth.cuh", "launch_cache.hpp")] + [
    os.path.join(os.path.dirname(HERE), "include", "daf.h")]

CU_SOURCES = ["api.cu", "compress.cu", "compress_stream_f32.cu", "compress_stream_f16.cu", "compress_stream_bf16.cu", "compress_twowidth_f32.cu", "compress_twowidth_f16.cu", "compress_twowidth_bf16.cu", "compress_twopass_f32.cu", "compress_twopass_f16.cu", "compress_twopass_bf16.cu", "compress_general_f32.cu", "compress_general_f16.cu",
              "compress_general_bf16.cu", "decompress.cu", "group_offsets.cu", "tensorwise.cu"]
CXX_SOURCES = ["pool.cpp", "store.cpp"]

# No fast-math, no flush-to-zero, no fused contraction beyond what the sources write out:
# results must match IEEE binary32 arithmetic bit for bit.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "--fmad=false", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


# Extra compiler flags for development builds (e.g. -DDAF_STAMPS), read when the library is built.
NVCC_FLAGS += os.environ.get("DAF_NVCC_EXTRA", "").split()


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    jobs = []
    for src in CU_SOURCES + CXX_SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ, src + ".o")
        if force or _stale(obj, [path] + HEADERS):
            jobs.append((src, [nvcc, *NVCC_FLAGS, "-c", path, "-o", obj]))

    def run(job):
        name, cmd = job
        r = subprocess.run(cmd, capture_output=True, text=True)
        with open(os.path.join(OBJ, name + ".log"), "w") as f:
            f.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {name}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            print(r.stdout + r.stderr)

    with ThreadPoolExecutor(max(1, min(len(jobs), os.cpu_count() or 1))) as ex:
        list(ex.map(run, jobs))
    objs = [os.path.join(OBJ, s + ".o") for s in CU_SOURCES + CXX_SOURCES]
    if force or jobs or _stale(LIB, objs):
        subprocess.check_call([nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
