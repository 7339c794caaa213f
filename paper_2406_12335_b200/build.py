"""Builds libvatp.so (sm_100a) in-tree with nvcc.  `python -m paper_2406_12335_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libvatp.so")
LIB_DEBUG = os.path.join(HERE, "libvatp_dbg.so")      # the bounds-checking build (-DVATP_DEBUG_BOUNDS)
SOURCES = ["vatp_api.cu", "prefill_simt.cu", "prefill_tc.cu", "prefill_static.cu", "attn_fwd.cu", "select.cu", "compact.cu", "window_ring.cu", "decode.cu", "decode_mma.cu", "decode_gqa.cu", "selftest.cu"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "vatp.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """debug_bounds: build libvatp_dbg.so instead, whose kernels range-check every index they compute and report
    a violation as VATP_ERR_BOUNDS in the status word (load it by setting VATP_LIBRARY to its path)."""
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and not is_stale(lib):
        return lib
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I", INCLUDE, "-shared", "-Xcompiler", "-fPIC", "-o", lib]
    if debug_bounds:
        cmd += ["-DVATP_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
