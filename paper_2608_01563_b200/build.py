"""Builds ``libmgn_attn.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2608_01563_b200.build [--force]
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libmgn_attn.so")
SOURCES = ["api.cu", "tmap.cu", "bwd_pre.cu", "strict_fwd.cu", "strict_bwd.cu", "strict_dq.cu", "fast_fwd.cu", "fast_fwd_small.cu", "fast_bwd.cu", "fast_dq.cu", "noalloc.cu", "peaks.cu", "selftest.cu", "proj.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
    "-DMGN_BUILD_SELFTEST=1",   # the bounded-wait self-test kernel (csrc/selftest.cu); no product path uses it
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _deps_mtime() -> float:
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    files.append(os.path.join(os.path.dirname(HERE), "include", "mgn_attn.h"))
    return max(os.path.getmtime(f) for f in files)


def _compile(src: str) -> str:
    obj = os.path.join(OBJ, src.replace(".cu", ".o"))
    log = obj + ".log"
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
    with open(log, "w") as fh:
        rc = subprocess.call(cmd, stdout=fh, stderr=subprocess.STDOUT)
    if rc != 0:
        sys.stderr.write(open(log).read())
        raise RuntimeError(f"nvcc failed on {src}")
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _deps_mtime():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(_compile, SOURCES))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs])
    os.replace(tmp, LIB)
    if verbose:
        for o in objs:
            for line in open(o + ".log"):
                if "registers" in line or "spill" in line or "Compiling entry" in line:
                    print(line.rstrip())
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
