"""Builds the C-ABI library of sm_100a kernels in-tree with nvcc."""

from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libnpd.so")
SOURCES = [os.path.join(HERE, "csrc", "npd_api.cu")]
DEPS = [os.path.join(HERE, "csrc", f) for f in
        ("npd_api.cu", "ptx_sm100.cuh", "gemm_sm100.cuh", "kd_tile_sm100.cuh", "small_kernels.cuh")]
DEPS.append(os.path.join(os.path.dirname(HERE), "include", "npd.h"))


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return cand


STAMP_PATH = LIB_PATH + ".sources"   # digest of the sources the library was built from


def sources_digest() -> str:
    h = hashlib.sha256()
    for d in sorted(DEPS):
        with open(d, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def is_stale() -> bool:
    """True when there is no library or it was built from other sources (by content, not by
    time stamps: a copied tree does not keep them in order)."""
    if not (os.path.exists(LIB_PATH) and os.path.exists(STAMP_PATH)):
        return True
    with open(STAMP_PATH) as f:
        return f.read().strip() != sources_digest()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libnpd.so for sm_100a if it is missing or older than its sources."""
    if not force and not is_stale():
        return LIB_PATH
    # nvcc writes to a name of its own and the finished file is moved into place, so that a
    # process loading the library at the same moment never sees half of it
    tmp = f"{LIB_PATH}.{os.getpid()}.tmp"
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
           "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-o", tmp] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if os.path.exists(STAMP_PATH):
        os.remove(STAMP_PATH)          # no stamp while the library and the stamp could disagree
    os.replace(tmp, LIB_PATH)
    with open(STAMP_PATH + ".tmp", "w") as f:
        f.write(sources_digest() + "\n")
    os.replace(STAMP_PATH + ".tmp", STAMP_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
