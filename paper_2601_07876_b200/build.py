"""Builds ``libnovak.so`` (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libnovak.so")
SOURCES = [os.path.join(CSRC, "novak_host.cpp"), os.path.join(CSRC, "novak_kernels.cu")]
HEADERS = [os.path.join(CSRC, "novak_internal.h"), os.path.join(ROOT, "include", "novak.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the NOVAK library cannot be built")


def nvcc_command(out: str = LIB, extra: list[str] | None = None) -> list[str]:
    return [
        nvcc_path(), "-O3", "-std=c++17",
        "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
        "-Xcompiler", "-fPIC,-Wall,-Wextra", "-shared",
        "-I", os.path.join(ROOT, "include"), "-I", CSRC,
        *(extra or []),
        "-o", out, *SOURCES,
    ]


def up_to_date(out: str = LIB) -> bool:
    if not os.path.exists(out):
        return False
    t = os.path.getmtime(out)
    return all(os.path.getmtime(f) <= t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, extra: list[str] | None = None) -> str:
    """Compiles the library if a source is newer than the built file."""
    if not force and not extra and up_to_date():
        return LIB
    tmp = f"{LIB}.{os.getpid()}.tmp"
    cmd = nvcc_command(tmp, (["-Xptxas", "-v"] if verbose else []) + (extra or []))
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed building libnovak.so")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
