"""Builds ``libthemis.so`` (CUDA kernels + C ABI) for sm_100a with nvcc.

Run as ``python -m paper_2407_14843_b200.build`` or call ``build_library()``.
The library is written next to this file; nvcc cross-compiles without a GPU.
``--check-bounds`` (``build_library(check_bounds=True)``) writes a second library,
``libthemis_check.so``, in which the solver kernels range-check every index they
compute (see ``themis_bounds_check_report`` in ``include/themis_probe.h``).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libthemis.so")
CHECK_LIB_PATH = os.path.join(_PKG, "libthemis_check.so")
SOURCES = sorted(glob.glob(os.path.join(_PKG, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(_PKG, "csrc", "*.h")) + glob.glob(os.path.join(_PKG, "csrc", "*.cuh"))) + [os.path.join(_ROOT, "include", "themis.h")]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _source_digest(check_bounds: bool) -> str:
    """Digest of everything a library is built from (sources, headers, the variant)."""
    import hashlib
    h = hashlib.sha256(b"check" if check_bounds else b"plain")
    for f in SOURCES + HEADERS:
        h.update(os.path.basename(f).encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def is_stale(path: str = LIB_PATH) -> bool:
    """True if the library is missing or was built from other sources.  The digest of its
    sources is kept beside it (file times do not survive a copy of the tree)."""
    try:
        with open(path + ".sha256") as fh:
            recorded = fh.read().strip()
    except OSError:
        return True
    return not os.path.exists(path) or recorded != _source_digest(path == CHECK_LIB_PATH)


def build_library(force: bool = False, verbose: bool = False, check_bounds: bool = False) -> str:
    """Compile the library (or its bounds-checked variant) if a source is newer than it;
    returns its path."""
    path = CHECK_LIB_PATH if check_bounds else LIB_PATH
    if not force and not is_stale(path):
        return path
    tmp = path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-Xcompiler", "-fno-gnu-unique", "-shared", "-Xptxas", "-v"] + (["-DTHEMIS_CHECK_BOUNDS", "-diag-suppress", "177"] if check_bounds else []) + [
           "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_PKG, "csrc"), "-o", tmp] + SOURCES
    proc = subprocess.run(cmd, capture_output=True, text=True)
    log = proc.stdout + proc.stderr
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + log)
    os.replace(tmp, path)
    with open(path + ".sha256", "w") as fh:
        fh.write(_source_digest(check_bounds) + "\n")
    if verbose:
        print(log)
    return path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True, check_bounds="--check-bounds" in sys.argv))
