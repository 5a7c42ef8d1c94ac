"""Builds libscout_b200.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libscout_b200.so")
SOURCES = ["scout_api.cu", "scout_sign.cu", "scout_one_launch.cu", "scout_noalloc.cu", "scout_vote.cu", "scout_timing.cu", "scout_ledger.cpp"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "-Xcompiler", "-fvisibility=hidden", "-Xlinker", "--exclude-libs,ALL"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def sources():
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    deps = srcs + [os.path.join(CSRC, h) for h in ("scout_internal.h", "scout_vote_device.cuh", "scout_scan.cuh", "scout_combine.cuh")] + \
        [os.path.join(ROOT, "include", h) for h in sorted(os.listdir(os.path.join(ROOT, "include")))]
    return srcs, deps


def is_stale() -> bool:
    _, deps = sources()
    return (not os.path.exists(LIB)) or os.path.getmtime(LIB) < max(os.path.getmtime(d) for d in deps)


def build(force: bool = False, verbose: bool = False, out: str = LIB, defines=()) -> str:
    """Compile the library.  ``out``/``defines`` build an alternative copy with
    other -D settings (select it at run time with the SCOUT_LIB variable)."""
    srcs, _ = sources()
    if out == LIB and not force and not is_stale():
        return LIB
    tmp = out + ".tmp%d" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-D" + d for d in defines] + \
          ["-I", os.path.join(ROOT, "include"), "-I", CSRC, "-shared", "-o", tmp] + srcs
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
