"""Builds libdash_attn.so (sm_100a only) in-tree with nvcc.  `python -m paper_2605_18753_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libdash_attn.so")
LIB_DEBUG = os.path.join(PKG, "libdash_attn_debug.so")
# translation units whose kernels index memory with values read from device memory: rebuilt with -DDASH_DEBUG
# (bounds checks that record DASH_ERR_CAPACITY instead of making the access) for the debug library
DEBUG_SOURCES = ["decode.cu", "decode_sm100.cu"]
OBJ_DIR = os.path.join(PKG, "build")
SOURCES = ["api.cu", "summaries.cu", "select.cu", "select_sm100.cu", "select_decode.cu", "attend_generic.cu", "attend_bwd_generic.cu", "route_bwd_generic.cu", "decode.cu", "decode_sm100.cu", "prefill_sm100.cu", "prefill_bwd_sm100.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the DashAttention library cannot be built")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libdash_attn.so; with debug=True also libdash_attn_debug.so (same library, bounds checks compiled in)."""
    nvcc = _nvcc()
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(ROOT, "include", "dash_attn.h"))
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src, dbg=False):
        obj = os.path.join(OBJ_DIR, ("debug_" if dbg else "") + src.replace(".cu", ".o"))
        path = os.path.join(CSRC, src)
        if force or _stale(obj, [path] + headers):
            cmd = [nvcc, *NVCC_FLAGS, *extra, *(["-DDASH_DEBUG"] if dbg else []), "-c", path, "-o", obj]
            res = subprocess.run(cmd, capture_output=True, text=True)
            if res.returncode != 0:
                raise RuntimeError(f"nvcc failed for {src}:\n{res.stdout}\n{res.stderr}")
            if verbose:
                sys.stderr.write(res.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
        dbg_objs = list(ex.map(lambda s_: compile_one(s_, True), DEBUG_SOURCES)) if debug else []

    def link(target, objects):
        if force or _stale(target, objects):
            cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", target, *objects]
            res = subprocess.run(cmd, capture_output=True, text=True)
            if res.returncode != 0:
                raise RuntimeError(f"link failed:\n{res.stdout}\n{res.stderr}")

    link(LIB, objs)
    if debug:
        swapped = {os.path.join(OBJ_DIR, s_.replace(".cu", ".o")): o for s_, o in zip(DEBUG_SOURCES, dbg_objs)}
        link(LIB_DEBUG, [swapped.get(o, o) for o in objs])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
