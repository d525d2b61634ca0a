"""Compile the CUDA kernels and the C ABI into ``libdart.so`` next to this file (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdart.so")
SOURCES = ["api.cu", "tmap.cu", "umma_gemm.cu", "umma_own.cu", "umma_dense.cu", "stage_inputs.cu", "attention.cu", "attn_umma.cu", "lm_head.cu", "topk_merge.cu", "topk_static.cu", "ngram_trie.cu", "tree.cu", "train_attn.cu", "selftest.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-DNDEBUG",
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "dart.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


LIB_DEBUG = os.path.join(HERE, "libdart_debug.so")


def build_debug(force: bool = False) -> str:
    """The same library with -DDART_DEBUG: index checks in front of the kernels' stores that record an error in
    the status word instead of writing out of range (what the GPU tests run once in place of a memory sanitizer)."""
    return build(force=force, lib=LIB_DEBUG, extra=["-DDART_DEBUG"], objdir="build_debug")


def build(force: bool = False, verbose: bool = False, lib: str = LIB, extra=(), objdir: str = "build") -> str:
    """Build libdart.so if it is missing or older than its sources; returns its path."""
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    os.makedirs(os.path.join(HERE, objdir), exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(HERE, objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    link = [nvcc, "-shared", "-o", lib, *objs, "-gencode", "arch=compute_100a,code=sm_100a", "-lcudart"]
    r = subprocess.run(link, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout)
        raise RuntimeError("link failed")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
