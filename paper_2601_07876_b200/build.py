"""Builds ``libnovak.so`` (the C-ABI library) in-tree with nvcc for sm_100a.

Every source is compiled to an object on its own, in parallel, then linked."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
import tempfile
import zlib
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libnovak.so")
# Gradient pre-processing modes of the step kernel (PRE_NONE / PRE_SCALE / PRE_CENTER /
# PRE_CENTER_ROWS, | 4 with a bf16 parameter copy, | 8 with bf16 moments): novak_step_inst.cu is compiled
# once per mode, and once more per mode for the graph-capturable kernel.
PRE_MODES = tuple(range(16))
DYN_PRE_MODES = (0, 1, 2, 4, 5, 6, 8, 9, 10, 12, 13, 14)   # no row-owning form (mode 3)
PLAIN_SOURCES = ("novak_host.cpp", "novak_host_device.cpp", "novak_host_step.cpp", "novak_launch.cu", "novak_launch_adapt.cu",
                 "novak_grad_stats.cu", "novak_trust_stats.cu", "novak_nesterov.cu", "novak_dyn.cu")
# (source, object name, extra flags)
UNITS = [(os.path.join(CSRC, f), f + ".o", []) for f in PLAIN_SOURCES]
UNITS += [(os.path.join(CSRC, "novak_step_inst.cu"), f"novak_step_mode{m}.o",
           [f"-DNOVAK_PRE_MODE={m}"]) for m in PRE_MODES]
UNITS += [(os.path.join(CSRC, "novak_step_inst.cu"), f"novak_step_dyn_mode{m}.o",
           [f"-DNOVAK_PRE_MODE={m}", "-DNOVAK_INST_DYN"]) for m in DYN_PRE_MODES]
ADAPT_PRE_MODES = DYN_PRE_MODES     # layer adaptation and update in one launch: no row-owning form either
UNITS += [(os.path.join(CSRC, "novak_step_inst.cu"), f"novak_step_adapt_mode{m}.o",
           [f"-DNOVAK_PRE_MODE={m}", "-DNOVAK_INST_ADAPT"]) for m in ADAPT_PRE_MODES]
SOURCES = sorted({u[0] for u in UNITS})
HEADERS = [os.path.join(CSRC, "novak_internal.h"), os.path.join(CSRC, "novak_handle.h"), os.path.join(CSRC, "novak_plan.h"),
           os.path.join(CSRC, "novak_step_types.h"),
           os.path.join(CSRC, "novak_step_kernel.cuh"), os.path.join(CSRC, "novak_step_dyn.cuh"),
           os.path.join(CSRC, "novak_trust.cuh"), os.path.join(CSRC, "novak_step_adapt.cuh"),
           os.path.join(ROOT, "include", "novak.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the NOVAK library cannot be built")


def compile_command(src: str, obj: str, extra: list[str] | None = None) -> list[str]:
    return [
        nvcc_path(), "-O3", "-std=c++17",
        "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
        "-Xcompiler", "-fPIC,-Wall,-Wextra",
        "-I", os.path.join(ROOT, "include"), "-I", CSRC,
        *(extra or []),
        "-x", "cu", "-c", "-o", obj, src,
    ]


def link_command(objs: list[str], out: str) -> list[str]:
    return [nvcc_path(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
            "-o", out, *objs]


def up_to_date(out: str = LIB) -> bool:
    if not os.path.exists(out):
        return False
    t = os.path.getmtime(out)
    return all(os.path.getmtime(f) <= t for f in SOURCES + HEADERS + [os.path.abspath(__file__)])


# objects and their dependency lists, kept between builds (outside the source tree: the
# tree is what gets copied around, and the objects are as large as the library)
OBJ_CACHE = os.path.join(tempfile.gettempdir(), "novak_build_%08x" % (zlib.crc32(PKG.encode()) & 0xffffffff))


def _object_is_current(obj: str, flags_key: str) -> bool:
    """An object is reused when it is newer than every file its last compilation read
    (nvcc's dependency list) and was compiled with the same flags."""
    dep, key = obj + ".d", obj + ".flags"
    if not (os.path.exists(obj) and os.path.exists(dep) and os.path.exists(key)):
        return False
    if open(key).read() != flags_key:
        return False
    t = os.path.getmtime(obj)
    text = open(dep).read().replace("\\\n", " ")
    files = text.split(":", 1)[1].split() if ":" in text else []
    return bool(files) and all(os.path.exists(f) and os.path.getmtime(f) <= t for f in files)


def build(force: bool = False, verbose: bool = False, extra: list[str] | None = None,
          out: str = LIB) -> str:
    """Compiles the library if a source is newer than the built file.  Objects are kept
    in a cache directory under the system's temporary directory with nvcc's dependency lists, so that a later build recompiles only the
    units whose sources changed; force=True recompiles everything."""
    if not force and not extra and out == LIB and up_to_date():
        return LIB
    flags = (["-Xptxas", "-v"] if verbose else []) + (extra or [])
    os.makedirs(OBJ_CACHE, exist_ok=True)
    objs = [os.path.join(OBJ_CACHE, u[1]) for u in UNITS]

    def one(pair):
        unit, obj = pair
        cmd = compile_command(unit[0], obj, flags + unit[2] + ["-MD", "-MF", obj + ".d"])
        key = " ".join(cmd)
        if not force and not verbose and _object_is_current(obj, key):
            return None
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode == 0:
            with open(obj + ".flags", "w") as f:
                f.write(key)
        elif os.path.exists(obj):
            os.remove(obj)
        return res

    with ThreadPoolExecutor(max_workers=len(UNITS)) as pool:
        results = [r for r in pool.map(one, zip(UNITS, objs)) if r is not None]
    failed = [r for r in results if r.returncode != 0]
    if verbose or failed:
        for r in results:
            sys.stderr.write(r.stdout + r.stderr)
    if failed:
        raise RuntimeError("nvcc failed building libnovak.so")
    tmp = f"{out}.{os.getpid()}.tmp"
    res = subprocess.run(link_command(objs, tmp), capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed linking libnovak.so")
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv))
