"""Build the CUDA library in-tree: ``python -m paper_2606_10944_b200.build [--force] [-v]``.

Every ``csrc/*.cu`` file is compiled for sm_100a (one nvcc per file, in parallel) and linked into
``csrc/libelm.so``.  A second library, ``csrc/libelm_check.so``, is the same code compiled with
``-DELM_BOUNDS_CHECK``: caller-supplied row numbers are checked on the device and a bad one is
reported through the call's status word instead of being read (a debugging aid; the tests use it
to show that the check reports and does not trap).
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

CSRC = Path(__file__).resolve().parent / "csrc"
LIB = CSRC / "libelm.so"
LIB_CHECK = CSRC / "libelm_check.so"
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def sources():
    return sorted(CSRC.glob("*.cu"))


def _deps():
    return list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [CSRC.parent.parent / "include" / "elm.h"]


def up_to_date(lib: Path = LIB) -> bool:
    if not lib.exists():
        return False
    t = lib.stat().st_mtime
    return all(d.stat().st_mtime <= t for d in _deps())


def _build_one(lib: Path, extra, verbose: bool) -> Path:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    objdir = CSRC / "build" / lib.stem
    objdir.mkdir(parents=True, exist_ok=True)

    def compile_one(src: Path) -> Path:
        obj = objdir / (src.stem + f".{os.getpid()}.o")
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", str(src), "-o", str(obj)]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.run(cmd, check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.run([nvcc, *NVCC_FLAGS[:2], "-shared", "-o", str(tmp), *map(str, objs)], check=True)
    os.replace(tmp, lib)
    for o in objs:
        o.unlink(missing_ok=True)
    return lib


def build(force: bool = False, verbose: bool = False, check_variant: bool = True) -> Path:
    extra = os.environ.get("ELM_NVCC_EXTRA", "").split()
    if force or not up_to_date(LIB):
        _build_one(LIB, extra, verbose)
    if check_variant and (force or not up_to_date(LIB_CHECK)):
        _build_one(LIB_CHECK, [*extra, "-DELM_BOUNDS_CHECK"], False)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
