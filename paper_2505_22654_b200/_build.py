"""Builds libvscan.so (sm_100a) in-tree with nvcc.  No torch types cross the boundary, so the
library is a plain shared object loaded with ctypes."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB_PATH = os.path.join(HERE, "libvscan.so")

STAMP_PATH = LIB_PATH + ".digest"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default", "-cudart", "static"]


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _deps():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC)) + [os.path.join(INCLUDE, "vscan.h")]


def source_digest() -> str:
    """Digest of everything the library is built from (file names and contents, build flags)."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for path in _deps():
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _stale() -> bool:
    """True when libvscan.so is missing or was built from other sources than the ones on disk.  The
    digest recorded next to the library decides, not file times (a copied tree has arbitrary ones)."""
    if not os.path.exists(LIB_PATH) or not os.path.exists(STAMP_PATH):
        return True
    with open(STAMP_PATH) as f:
        return f.read().strip() != source_digest()


def have_nvcc() -> bool:
    return os.path.exists(shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc")


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ into one shared library next to this file."""
    if not force and not _stale():
        return LIB_PATH
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: libvscan.so cannot be built")
    digest = source_digest()
    cmd = [nvcc, "-shared", "-o", LIB_PATH, "-I", INCLUDE, "-I", CSRC] + NVCC_FLAGS
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += sources()
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    with open(STAMP_PATH, "w") as f:
        f.write(digest + "\n")
    if verbose:
        sys.stderr.write(res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
