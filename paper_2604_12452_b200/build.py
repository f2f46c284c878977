"""In-tree build of the CUDA library (liblca.so) for sm_100a with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "liblca.so")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON = ARCH + ["-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
# The attention kernels use the approximate exponentials / reciprocals on purpose (their results are
# rounded to bf16 probabilities and outputs); the condensation keeps IEEE arithmetic: its softmax
# weights and pooled sums are compared with the oracle at one bf16 ulp.
SOURCES = {
    "lca_api.cu": [],
    "condense.cu": [],
    "attn_simt.cu": ["--use_fast_math"],
    "attn_tc.cu": ["--use_fast_math"],
    "attn_tc2.cu": ["--use_fast_math"],
    "attn_gqa2.cu": ["--use_fast_math"],
    "gemm_uv.cu": ["--use_fast_math"],
}


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(PKG), "include", "lca.h"))
    deps.append(os.path.abspath(__file__))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu to an object (in parallel) and link one shared library next to the
    package.  Returns its path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ, exist_ok=True)
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(item):
        src, flags = item
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        subprocess.check_call([nvcc] + COMMON + flags + extra + ["-c", os.path.join(CSRC, src), "-o", obj])
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES.items()))
    subprocess.check_call([nvcc] + ARCH + ["-shared", "-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
