"""Builds liblsa.so (hand-written sm_100a CUDA behind the C ABI of include/lsa.h) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "liblsa.so")
SOURCES = ["lsa_api.cu", "lsa_index.cu", "lsa_attn.cu", "lsa_static.cu", "lsa_coarse_tc.cu", "lsa_attn_tc.cu", "lsa_fine_tc.cu",
           "lsa_coarse_paged_tc.cu", "lsa_fine_big_tc.cu", "lsa_scores_paged_tc.cu", "lsa_fine_paged_tc.cu", "lsa_selftest.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh", ".h"))]
    deps.append(os.path.join(ROOT, "include", "lsa.h"))
    return any(os.path.getmtime(d) > t for d in deps)


CHECK_LIB_PATH = os.path.join(PKG_DIR, "liblsa_check.so")


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Compile every CUDA source for sm_100a and link liblsa.so; returns its path.

    check=True builds the checking variant liblsa_check.so instead (-DLSA_CHECK: the attention kernels validate
    caller-given cache row numbers and report LSA_ERR_INDEX instead of reading outside the cache); load it by
    setting LSA_LIBRARY to its path before the first call into the binding."""
    if check:
        if not force and not _stale(CHECK_LIB_PATH):
            return CHECK_LIB_PATH
        return _build_to(CHECK_LIB_PATH, ["-DLSA_CHECK"], "_check.o", verbose)
    if not force and not _stale():
        return LIB_PATH
    return _build_to(LIB_PATH, [], ".o", verbose)


def _build_to(lib_path: str, extra: list, obj_suffix: str, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", obj_suffix))
        cmd = [nvcc, *NVCC_FLAGS, *extra, *os.environ.get("LSA_NVCC_EXTRA", "").split(), "-Xcompiler", "-DLSA_BUILDING=1", "-c",
               os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode != 0:
            sys.stderr.write(out)
        if pr.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    link = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib_path, *objs, "-lcudart"]
    subprocess.run(link, check=True)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, check="--check" in sys.argv))
