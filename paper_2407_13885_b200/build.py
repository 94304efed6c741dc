"""Builds ``libattnw.so`` in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libattnw.so")
SOURCES = [os.path.join(_CSRC, "attnw_api.cu")]
_DEPS = [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC))] + [
    os.path.join(os.path.dirname(_PKG), "include", "attnw.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; it is needed to build libattnw.so")


def nvcc_command(out: str, verbose_ptxas: bool = False, defines: tuple[str, ...] = ()) -> list[str]:
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", out, *SOURCES]
    if verbose_ptxas:
        cmd[1:1] = ["-Xptxas", "-v"]
    for d in defines:
        cmd.insert(1, "-D" + d)
    return cmd


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > built for d in _DEPS)


def build_library(force: bool = False, verbose_ptxas: bool = False, defines: tuple[str, ...] = (),
                  out: str | None = None) -> str:
    """Compile if the library is missing or older than its sources; returns its path.  `defines` and `out` build a
    variant beside the product library (the instrumented build of timeline.py); the product library has none."""
    target = out or LIB_PATH
    if defines and out is None:
        raise ValueError("a build with extra definitions needs its own output path")
    if not force and out is None and not is_stale():
        return LIB_PATH
    tmp = target + f".tmp{os.getpid()}"
    proc = subprocess.run(nvcc_command(tmp, verbose_ptxas, defines), capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout + proc.stderr)
    os.replace(tmp, target)
    if verbose_ptxas:
        print(proc.stderr)
    return target


if __name__ == "__main__":
    import sys
    print(build_library(force="--force" in sys.argv, verbose_ptxas="-v" in sys.argv))
