"""Builds libdscale.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdscale.so")
# The same sources with every device-side wait bounded at about 1 ms and a hook that leaves out one
# copy: what tests/test_gpu_wait_limit.py loads to make a bounded wait run out.  Never loaded by the package.
LIB_WAIT_TEST = os.path.join(HERE, "libdscale_waittest.so")
WAIT_TEST_FLAGS = ["-DDSCALE_WAIT_TEST", "-DDSCALE_WAIT_CYCLES=2000000LL"]
SOURCES = ["api.cu", "alloc.cu", "accept.cu", "accept_static.cu", "accept_sampling.cu", "attn_simt.cu", "attn_tc.cu", "attn_padded.cu", "lm_head.cu", "predictor.cu"]
FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(HERE, "..", "include", "dscale.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library (and its wait-limit test variant) if missing or older than the sources."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    for lib, extra in ((LIB, []), (LIB_WAIT_TEST, WAIT_TEST_FLAGS)):
        if not force and not _stale(lib):
            continue
        cmd = [nvcc] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + SOURCES
        res = subprocess.run(cmd, cwd=CSRC, capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("nvcc failed building " + os.path.basename(lib))
        if verbose:
            sys.stderr.write(res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
