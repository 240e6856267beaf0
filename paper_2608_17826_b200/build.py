"""Builds libbsr.so (the CUDA library behind include/bsr.h) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "bsr_lib.cu")
DEPS = [SRC, os.path.join(HERE, "csrc", "bsr_kernels.cuh"),
        os.path.join(os.path.dirname(HERE), "include", "bsr.h")]
LIB = os.path.join(HERE, "libbsr.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC,-O3,-pthread", "-Xptxas", "-v",
]


def nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the BSR library cannot be built")
    return exe


def up_to_date() -> bool:
    return os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in DEPS)


def _compile(out: str, defines: list[str], verbose: bool) -> str:
    # built under a private name and renamed into place: several processes of one job (one per GPU)
    # may find the library stale at the same moment, and none of them may load a half-written file
    tmp = f"{out}.{os.getpid()}.tmp"
    cmd = [nvcc(), *NVCC_FLAGS, *defines, "-o", tmp, SRC]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, out)
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    return _compile(LIB, [], verbose)


# A second build of the same source for the tests: the bulk install kernel with a ring of only
# three 1 KiB stages, one lagging store and at most 32 CTAs per launch, so that every shared-memory
# stage is recycled hundreds of times per CTA (the product build recycles a 16 KiB stage about ten
# times).  An ordering slip between a stage's store, its checksum and its next load has hundreds of
# chances per CTA to show as a wrong byte or sum here.
STRESS_LIB = os.path.join(HERE, "libbsr_stress.so")
STRESS_DEFINES = ["-DBSR_K_BULK_STAGES=3", "-DBSR_K_BULK_STORE_LAG=1", "-DBSR_K_TILE_MAX=1024u",
                  "-DBSR_K_BULK_TILES_PER_CTA=512", "-DBSR_K_BULK_MAX_GRID=32"]


def build_stress(force: bool = False, verbose: bool = False) -> str:
    fresh = os.path.exists(STRESS_LIB) and all(os.path.getmtime(STRESS_LIB) >= os.path.getmtime(d) for d in DEPS)
    if not force and fresh:
        return STRESS_LIB
    return _compile(STRESS_LIB, STRESS_DEFINES, verbose)


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build_stress(force=True))
