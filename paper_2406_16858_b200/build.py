"""Builds ``libeagle2.so`` in the package directory with nvcc for sm_100a.

    python -m paper_2406_16858_b200.build [--force]

The library links the CUDA runtime statically, so it loads (and its host-side argument checks run)
on a machine without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_PKG, "_build")
LIB_PATH = os.path.join(_PKG, "libeagle2.so")

SOURCES = ["api.cu", "expand.cu", "rerank_mask.cu", "tree_attention.cu", "accept.cu", "kv_compact.cu", "lm_head.cu", "lm_head_topk.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-I", os.path.join(_ROOT, "include"), "-I", _CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _newest_dep() -> float:
    deps = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)] + [os.path.join(_ROOT, "include", "eagle2.h")]
    return max(os.path.getmtime(p) for p in deps)


def _compile(src: str, force: bool, newest: float) -> tuple[str, str]:
    obj = os.path.join(_OBJ, src.replace(".cu", ".o"))
    log = ""
    if force or not os.path.exists(obj) or os.path.getmtime(obj) < newest:
        res = subprocess.run([_nvcc(), *NVCC_FLAGS, "-c", os.path.join(_CSRC, src), "-o", obj],
                             capture_output=True, text=True)
        log = res.stdout + res.stderr
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{log}")
    return obj, log


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(_OBJ, exist_ok=True)
    newest = _newest_dep()
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= newest:
        return LIB_PATH
    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        results = list(pool.map(lambda s: _compile(s, force, newest), SOURCES))
    if verbose:
        for _, log in results:
            if log:
                print(log)
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *[o for o, _ in results],
                           "-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
