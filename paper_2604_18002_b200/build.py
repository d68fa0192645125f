"""Builds the CUDA library in tree: nvcc for sm_100a only, one object per
translation unit, linked into ``libngc_b200.so`` beside this file.

    python -m paper_2604_18002_b200.build [--force] [--verbose] [--debug] [--nvtx]

``--debug`` builds a second library, ``libngc_b200_debug.so``, whose kernels check every index
they compute before using it and report a violation through the device status word (the
stand-in for a memory checker: the GPU tests rerun their small cases on it).  ``--nvtx`` wraps
every C-ABI call in an NVTX range so that profiler timelines name the call a kernel belongs
to; it can be combined with either build and changes nothing else.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libngc_b200.so")

SOURCES = ["api.cu", "compact_kv.cu", "sample_evict.cu", "evict_logprob.cu", "decode_attn.cu", "score_evict.cu", "replay_visibility.cu", "score_backward.cu", "score_backward_umma.cu", "replay_attn.cu", "replay_attn_umma.cu", "selftest.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC,
    # the sampling contract needs IEEE arithmetic: never --use_fast_math
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.exists(cand) or "/" not in cand):
            return cand
    raise RuntimeError("nvcc not found")


def _deps():
    hdrs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hdrs.append(os.path.join(INCLUDE, "ngc.h"))
    return hdrs


def build(force: bool = False, verbose: bool = False, debug: bool = False, nvtx: bool = False) -> str:
    variant = ("_debug" if debug else "") + ("_nvtx" if nvtx else "")
    obj_dir = OBJ_DIR + variant
    lib_path = LIB.replace(".so", variant + ".so")
    extra = (["-DNGC_DEBUG"] if debug else []) + (["-DNGC_NVTX"] if nvtx else [])
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    hdr_time = max(os.path.getmtime(h) for h in _deps())
    jobs = []
    objs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr_time):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    if jobs:
        with ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for out in ex.map(run, jobs):
                if verbose and out:
                    print(out)
    if jobs or not os.path.exists(lib_path):
        tmp = lib_path + f".tmp{os.getpid()}"
        run([nvcc, "-shared", "-o", tmp] + objs + ["-cudart", "static"] + (["-ldl"] if nvtx else []))
        os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv,
                nvtx="--nvtx" in sys.argv))
