"""Build the CUDA library (libmpfa.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmpfa.so")
SOURCES = ["quantize.cu", "prefill.cu", "prefill_pair.cu", "decode.cu", "api.cu", "mma_peak.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "mpfa.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", LIB,
               *[os.path.join(CSRC, s) for s in SOURCES]]
        subprocess.check_call(cmd)
    return LIB


# A second, test-only build of the same sources: bounded device waits of a few milliseconds instead of two seconds,
# and one shared-memory copy left out on purpose in CTA 0 (see MPFA_TEST_DROP_V_COPY in csrc/prefill_common.cuh), so
# that a GPU test can make a wait run out and watch the library give up cleanly.  Never loaded by the binding.
GIVEUP_TEST_LIB = os.path.join(HERE, "libmpfa_giveup_test.so")
GIVEUP_TEST_FLAGS = ["-DMPFA_WAIT_LIMIT_CYCLES=20000000ll", "-DMPFA_DRAIN_LIMIT_NS=10000000ull", "-DMPFA_TEST_DROP_V_COPY"]


def build_giveup_test_lib(force: bool = False) -> str:
    stale = not os.path.exists(GIVEUP_TEST_LIB) or any(
        os.path.getmtime(os.path.join(CSRC, f)) > os.path.getmtime(GIVEUP_TEST_LIB) for f in os.listdir(CSRC))
    if force or stale:
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, *NVCC_FLAGS, *GIVEUP_TEST_FLAGS, "-o", GIVEUP_TEST_LIB,
                               *[os.path.join(CSRC, s) for s in SOURCES]])
    return GIVEUP_TEST_LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
