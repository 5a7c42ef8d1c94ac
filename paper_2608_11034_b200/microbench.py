"""Builds and runs the two microbenchmarks behind the scan's compute bound.

    python -m paper_2608_11034_b200.microbench [sm_mhz]

pipe_rates: issue cost of the instruction kinds the row routine is made of, alone and
mixed.  row_cost: SM cycles per 512-byte row of the routine itself with its rows in shared
memory (no DRAM), per dtype, for the hash fold, the statistics and both.  Both need a GPU;
they print plain text.  ``sm_mhz`` is the clock the event times are converted with (default
1965, the maximum SM clock of a B200)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "microbench")
OUT = os.path.join(HERE, "microbench_bin")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
         "-I", os.path.join(os.path.dirname(HERE), "include"), "-I", os.path.join(HERE, "csrc")]


def build() -> list:
    os.makedirs(OUT, exist_ok=True)
    exes = []
    for name in ("pipe_rates", "row_cost"):
        exe = os.path.join(OUT, name)
        src = os.path.join(SRC, name + ".cu")
        deps = [src] + [os.path.join(HERE, "csrc", h) for h in ("scout_scan.cuh", "scout_internal.h")]
        if not os.path.exists(exe) or os.path.getmtime(exe) < max(os.path.getmtime(d) for d in deps):
            subprocess.check_call([os.environ.get("NVCC", "nvcc")] + FLAGS + ["-o", exe, src])
        exes.append(exe)
    return exes


if __name__ == "__main__":
    args = sys.argv[1:]
    only_build = "--build-only" in args
    args = [a for a in args if a != "--build-only"]
    for exe in build():
        if not only_build:
            print("==", os.path.basename(exe), flush=True)
            subprocess.check_call([exe] + args)
