"""Builds libdsn.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every translation unit is compiled on its own (in parallel, objects cached under _build/ by source
time stamp) and the objects are linked into one shared library.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
OBJ_DIR = os.path.join(PKG_DIR, "_build")
LIB_PATH = os.path.join(PKG_DIR, "libdsn.so")
SOURCES = ["dsn_api.cu", "dsn_gate.cu", "dsn_route.cu", "dsn_copy.cu", "dsn_linear_f32.cu", "dsn_gemm_bf16.cu",
           "dsn_gemm_bf16_2cta.cu", "dsn_gemm_bf16_chain.cu", "dsn_conv3x3_halo.cu", "dsn_attention.cu", "dsn_attention_ws.cu",
           "dsn_depthwise.cu", "dsn_dwpw.cu", "dsn_selftest.cu"]


def _headers_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    paths.append(os.path.join(ROOT, "include", "dsn.h"))
    return max(os.path.getmtime(p) for p in paths)


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "dsn.h")]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    hdr = _headers_mtime()

    def compile_one(src: str):
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ_DIR, src[:-3] + ".o")
        if (not force and not verbose and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(os.path.getmtime(path), hdr)):
            return obj, 0, ""
        res = subprocess.run([nvcc] + flags + ["-c", path, "-o", obj], capture_output=True, text=True)
        return obj, res.returncode, res.stdout + res.stderr

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        results = list(pool.map(compile_one, SOURCES))
    for src, (obj, rc, log) in zip(SOURCES, results):
        if verbose and log:
            sys.stderr.write(f"== {src}\n{log}")
        if rc != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{log}")
    res = subprocess.run([nvcc, "-shared", "-cudart", "shared", "-o", LIB_PATH] + [r[0] for r in results],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
