"""Builds ``libaibx_synth.so`` (the device and native-host twins of this package's generator,
and the memory-system probes the benchmark uses as measured ceilings) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
SRCS = [os.path.join(PKG, "csrc", f) for f in ("synth_fill.cu", "mem_probe.cu")]
SYNTH_LIB = os.path.join(PKG, "libaibx_synth.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def build(force: bool = False) -> None:
    if (not force and os.path.exists(SYNTH_LIB)
            and os.path.getmtime(SYNTH_LIB) >= max(os.path.getmtime(f) for f in SRCS)):
        return
    subprocess.check_call(["nvcc"] + NVCC_FLAGS + SRCS + ["-o", SYNTH_LIB + ".tmp"])
    os.replace(SYNTH_LIB + ".tmp", SYNTH_LIB)


if __name__ == "__main__":
    import sys

    build(force="--force" in sys.argv)
    print(SYNTH_LIB)
