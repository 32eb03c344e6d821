"""Builds the CUDA library in-tree: paper_2401_06104_b200/libtova.so (sm_100a only)."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_SRC_DIR = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libtova.so")
_STAMP = LIB_PATH + ".stamp"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--shared", "-Xcompiler", "-fPIC"]


def _sources():
    files = [os.path.join(_SRC_DIR, f) for f in sorted(os.listdir(_SRC_DIR))
             if f.endswith((".cu", ".cuh", ".h"))]
    files.append(os.path.join(_ROOT, "include", "tova.h"))
    return files


def _digest() -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for f in _sources():
        h.update(f.encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libtova.so unless an up-to-date build exists."""
    want = _digest()
    if not force and os.path.exists(LIB_PATH) and os.path.exists(_STAMP):
        with open(_STAMP) as fh:
            if fh.read().strip() == want:
                return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cus = [f for f in _sources() if f.endswith(".cu")]
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + cus
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    os.replace(tmp, LIB_PATH)
    with open(_STAMP, "w") as fh:
        fh.write(want)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
