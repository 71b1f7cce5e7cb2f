"""Build the CUDA library in-tree: csrc/*.cu -> paper_2510_26771_b200/libstamp.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libstamp.so")


def _sources():
    srcs = [os.path.join(_CSRC, "stamp_api.cu")]
    deps = [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC))] + [os.path.join(_ROOT, "include", "stamp.h")]
    return srcs, deps


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _sources()[1])


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile with nvcc for sm_100a.  Returns the path of the shared library."""
    if not force and not needs_build():
        return LIB_PATH
    srcs, _ = _sources()
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared",
           "-I", os.path.join(_ROOT, "include"), "-I", _CSRC, "-o", tmp] + srcs
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
