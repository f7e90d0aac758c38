"""Builds the CUDA library in-tree with nvcc for sm_100a (no other architecture: the int8
tensor-core path does not exist elsewhere)."""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libniti_b200.so")
SOURCES = ["niti_api.cu", "niti_elementwise.cu", "niti_simt_gemm.cu", "niti_tc_gemm.cu"]


def _newest_source() -> float:
    t = 0.0
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


def source_digest() -> str:
    """SHA-256 over the CUDA sources and the public header, in a fixed order."""
    h = hashlib.sha256()
    inc = os.path.join(os.path.dirname(HERE), "include")
    files = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))] + [os.path.join(inc, "niti.h")]
    for f in files:
        h.update(os.path.basename(f).encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def built_from_current_sources():
    """True / False when the library carries a record of the sources it was built from; None without one."""
    try:
        with open(LIB + ".sha256") as fh:
            return fh.read().strip() == source_digest()
    except OSError:
        return None


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB):
        same = built_from_current_sources()          # (no record: a build from before the record existed)
        if same is True or (same is None and os.path.getmtime(LIB) >= _newest_source()):
            return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", LIB + ".tmp"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(LIB + ".tmp", LIB)
    with open(LIB + ".sha256", "w") as fh:          # which sources this binary was built from
        fh.write(source_digest() + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
