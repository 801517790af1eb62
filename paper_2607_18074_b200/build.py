"""Builds libsobek.so (sm_100a) in-tree with nvcc: one object per source, compiled in parallel."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libsobek.so")
SOURCES = ["plan.cu", "graph.cu", "kernels.cu", "edge_stream.cu", "edge_stream_k8.cu", "edge_stream_k8d.cu",
           "edge_stream_k16.cu", "edge_stream_k16d.cu", "stream_tc.cu", "edge_pass.cu", "edge_pass_tc.cu", "fused.cu", "fused_k8.cu", "fused_k8d.cu", "fused_k16.cu", "fused_k16d.cu", "gemm_tc.cu", "node_uvu.cu", "uvu_direct.cu", "geometry_second.cu", "api.cu", "static_scratch.cu"]
FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC",
         "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + \
           [os.path.join(ROOT, "include", "sobek.h")]


def _compile(src: str, force: bool, verbose_ptxas: bool) -> str:
    obj = os.path.join(OBJ, src.replace(".cu", ".o"))
    path = os.path.join(CSRC, src)
    deps = [path] + _headers()
    if not force and os.path.exists(obj) and all(os.path.getmtime(d) <= os.path.getmtime(obj) for d in deps):
        return obj
    cmd = ["nvcc"] + FLAGS + (["-Xptxas", "-v"] if verbose_ptxas else []) + ["-c", path, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose_ptxas or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}")
    return obj


def build(force: bool = False, verbose_ptxas: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(lambda s: _compile(s, force, verbose_ptxas), SOURCES))
    if force or not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        subprocess.check_call(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    build(force="-f" in sys.argv, verbose_ptxas="-v" in sys.argv)
    print(LIB)
