"""Builds ``libsentinel.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB = os.path.join(_HERE, "libsentinel.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _inputs():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    files += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    files.append(os.path.abspath(__file__))          # a change of flags rebuilds too
    return files


LIB_CHECKED = os.path.join(_HERE, "libsentinel_checked.so")     # the same sources with -DSENTINEL_CHECK_BOUNDS


def _compile(target: str, extra: list, force: bool, verbose: bool) -> str:
    newest = max(os.path.getmtime(f) for f in _inputs())
    if not force and os.path.exists(target) and os.path.getmtime(target) >= newest:
        return target
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = target + ".tmp%d" % os.getpid()
    cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", INCLUDE, "-I", CSRC, "-o", tmp, *_sources()]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, target)
    return target


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ into one shared library; returns its path."""
    return _compile(LIB, [], force, verbose)


def build_checked(force: bool = False, verbose: bool = False) -> str:
    """The checked build: every index derived from the shape is compared with its buffer's extent
    before the access (a debugging aid; the kernels are slower)."""
    return _compile(LIB_CHECKED, ["-DSENTINEL_CHECK_BOUNDS"], force, verbose)


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build_checked(force=True))
