"""Builds the C-ABI CUDA library in-tree: paper_2602_01801_b200/lib/libfastar.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libfastar.so")
# the range-checking build (-DFASTAR_DEBUG_BOUNDS): computed slot / block / page / token indices are checked on the
# device, a violation is recorded in the status word and the access redirected; used by tests/test_gpu_debug_bounds.py
BOUNDS_LIB_PATH = os.path.join(LIB_DIR, "libfastar_bounds.so")
# host code under AddressSanitizer + UndefinedBehaviorSanitizer (device code unchanged); loaded by a CPU test in a
# child process that preloads the sanitizer runtime
SAN_LIB_PATH = os.path.join(LIB_DIR, "libfastar_hostsan.so")
SAN_FLAGS = ["-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined", "-Xcompiler", "-fno-omit-frame-pointer",
             "-Xcompiler", "-fno-sanitize-recover=undefined"]
SOURCES = ["gemm_kernels.cu", "attn_kernels.cu", "update_kernels.cu", "commit_kernel.cu", "search8_kernels.cu", "fastar_api.cu", "noalloc_select.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug_bounds: bool = False, host_sanitizers: bool = False) -> str:
    os.makedirs(LIB_DIR, exist_ok=True)
    obj_dir = os.path.join(LIB_DIR, "obj_hostsan" if host_sanitizers else "obj_bounds" if debug_bounds else "obj")
    lib_path = SAN_LIB_PATH if host_sanitizers else BOUNDS_LIB_PATH if debug_bounds else LIB_PATH
    extra = (["-DFASTAR_DEBUG_BOUNDS"] if debug_bounds else []) + (SAN_FLAGS if host_sanitizers else [])
    os.makedirs(obj_dir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "fastar.h"))
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    nvcc = _nvcc()

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        path = os.path.join(CSRC, src)
        if force or _stale(obj, [path] + headers):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", path, "-o", obj]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose:
                sys.stderr.write(r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        return obj

    with ThreadPoolExecutor(max_workers=4) as ex:
        objs = list(ex.map(compile_one, sources))
    if force or _stale(lib_path, objs):
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path] + objs
        if host_sanitizers:
            cmd += ["-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--hostsan" in sys.argv:
        print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, host_sanitizers=True))
    if "--bounds" in sys.argv:
        print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds=True))
