"""Builds libtasc.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libtasc.so")
SOURCES = ["api.cu", "drafter.cu", "gemm_tcgen05.cu", "gemm_fused.cu", "gemm_wide.cu", "attention_mma.cu", "gemm_simt.cu", "gemm_static.cu", "tasc_tok.cu", "layers.cu", "attention.cu", "profile.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]


def _newer(src: str, dst: str) -> bool:
    return not os.path.exists(dst) or os.path.getmtime(src) > os.path.getmtime(dst)


def build_timeline() -> str:
    """Builds libtasc_timeline.so: the same sources with -DTASC_TIMELINE (per-CTA time stamps on the global
    timer, read by paper_2602_24174_b200.timeline).  Relocatable device code, because the log is one device
    symbol shared by several translation units.  A development aid; the product library has none of it."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    out = os.path.join(HERE, "libtasc_timeline.so")
    objs, procs = [], []
    for src in SOURCES:
        o = os.path.join(CSRC, src[:-3] + ".tl.o")
        objs.append(o)
        cmd = [nvcc, *NVCC_FLAGS, "-rdc=true", "-DTASC_TIMELINE", "-c", os.path.join(CSRC, src), "-o", o]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out_text, _ = p.communicate()
        if p.returncode != 0:
            sys.stderr.write(f"--- {src}\n{out_text}\n")
            failed = True
    if failed:
        raise RuntimeError("nvcc failed")
    subprocess.check_call([nvcc, "-shared", "-rdc=true", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-o", out, *objs, "-lcudart"])
    for o in objs:
        os.remove(o)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(INCLUDE, "tasc.h"))
    objs, procs = [], []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src[:-3] + ".o")
        objs.append(o)
        if force or _newer(s, o) or any(_newer(h, o) for h in headers):
            cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-c", s, "-o", o]
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or not os.path.exists(LIB):
        subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB, *objs, "-lcudart"])
    return LIB


if __name__ == "__main__":
    if "--timeline" in sys.argv:
        print(build_timeline())
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
