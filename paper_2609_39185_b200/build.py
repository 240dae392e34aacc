"""Build libssdq.so (the C-ABI CUDA library) in-tree for sm_100a with nvcc.

Usage: python -m paper_2609_39185_b200.build [--force] [--verbose] [--debug]
One object per translation unit, compiled in parallel, then linked with a static CUDA runtime.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libssdq.so")
OBJ_DIR = os.path.join(HERE, "build")

SOURCES = ["ssdq_api.cu", "ssdq_update_fp16.cu", "ssdq_update_bf16.cu", "ssdq_update_e4m3.cu", "ssdq_update_fp32.cu", "ssdq_update_int8.cu",
           "ssdq_quantize.cu", "ssdq_metrics.cu"]
# --fmad=false: nothing is contracted behind the kernels' backs; every fused multiply-add is written out.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "--fmad=false",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include")]


def _newest_source_mtime():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "ssdq.h")]
    return max(os.path.getmtime(f) for f in files)


DEBUG_LIB = os.path.join(HERE, "libssdq_debug.so")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """debug=True builds libssdq_debug.so, the same sources with -DSSDQ_DEBUG (index-range checks in every update kernel)."""
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    lib_path = DEBUG_LIB if debug else LIB
    obj_dir = os.path.join(OBJ_DIR, "debug") if debug else OBJ_DIR
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= _newest_source_mtime():
        return lib_path
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

    def compile_one(src):
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        cmd = [nvcc] + NVCC_FLAGS + (["-DSSDQ_DEBUG"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            with open(obj.replace(".o", ".ptxas.txt"), "w") as f:
                f.write(r.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(sources))) as ex:
        objs = list(ex.map(compile_one, sources))
    cmd = [nvcc, "-shared", "-o", lib_path] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
