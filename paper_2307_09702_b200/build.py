"""Builds ``libfsmguide.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libfsmguide.so")
# The same sources with -DFSM_CHECKED: every index that depends on data is range-checked
# (FSM_FLAG_INDEX instead of a stray access).  A test aid, never the library the binding
# loads by default.
CHECKED_LIB_PATH = os.path.join(_PKG, "libfsmguide_checked.so")
SOURCES = ["fsm_api.cu", "fsm_index.cu", "fsm_index_alias.cu", "fsm_index_io.cu", "fsm_mask_step.cu"]
# No --use_fast_math: the decode step compares logits as IEEE floats, subnormals included
# (that flag flushes them to zero), and nothing on the path needs approximate division or
# transcendentals.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-ftz=false", "-prec-div=true", "-prec-sqrt=true", "-fmad=true",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(lib_path: str) -> bool:
    if not os.path.exists(lib_path):
        return True
    built = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "fsmguide.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def _compile(lib_path: str, extra: list[str], verbose: bool) -> None:
    tmp = lib_path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-I", INCLUDE, "-I", CSRC, "-shared", "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib_path)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library, and its range-checked twin, if missing or older than the sources."""
    if force or _stale(LIB_PATH):
        _compile(LIB_PATH, [], verbose)
    if force or _stale(CHECKED_LIB_PATH):
        _compile(CHECKED_LIB_PATH, ["-DFSM_CHECKED"], verbose)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
