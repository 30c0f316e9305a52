"""Builds librattn.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2506_15545_b200.build [--force]

Objects go to ``_build/`` (git-ignored); the shared library is written next to this
file so that it travels with the source tree.
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(ROOT, "_build")
LIB = os.path.join(HERE, "librattn.so")
LIB_DEBUG = os.path.join(HERE, "librattn_dbg.so")      # same sources with -DRATTN_DEBUG_KNOBS (include/rattn_debug.h)
LIB_TIMELINE = os.path.join(HERE, "librattn_tl.so")    # same sources with -DRATTN_TIMELINE (bench.py --case timeline)

SOURCES = ["rattn_api.cu", "generic_fwd.cu", "generic_bwd.cu", "decode.cu", "tc_fwd.cu",
           "tc_fwd2.cu", "tc_state.cu", "tc_bwd.cu", "static_scratch.cu", "qk_prologue.cu", "decode_tc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC",
              "-I" + os.path.join(ROOT, "include"), "-I" + CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _newest_dep_mtime() -> float:
    m = max(os.path.getmtime(os.path.join(ROOT, "include", f)) for f in ("rattn.h", "rattn_debug.h"))
    for f in os.listdir(CSRC):
        m = max(m, os.path.getmtime(os.path.join(CSRC, f)))
    return max(m, os.path.getmtime(__file__))


def _compile(src: str, verbose: bool, debug: bool = False, timeline: bool = False) -> str:
    obj = os.path.join(BUILD, src.replace(".cu", ".dbg.o" if debug else ".tl.o" if timeline else ".o"))
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
    if debug:
        cmd.insert(1, "-DRATTN_DEBUG_KNOBS")
    if timeline:
        cmd.insert(1, "-DRATTN_TIMELINE")
    if os.path.exists(os.path.join(CSRC, "tc_fwd.cu")):
        cmd.insert(1, "-DRATTN_HAVE_TC")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
    if verbose:
        sys.stderr.write(r.stderr)
    return obj


def build(force: bool = False, verbose: bool = False, debug: bool = False, timeline: bool = False) -> str:
    """Compile every source and link librattn.so (debug: librattn_dbg.so; timeline: librattn_tl.so,
    the forward kernel with its per-role clock stamps compiled in); returns its path."""
    lib = LIB_DEBUG if debug else LIB_TIMELINE if timeline else LIB
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_dep_mtime():
        return lib
    os.makedirs(BUILD, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(sources)) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose, debug, timeline), sources))
    cmd = [_nvcc(), "-shared", "-o", lib, *objs, "-cudart", "static"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build(force="--force" in sys.argv, debug=True))
