"""Builds ``liba2sf.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2407_20485_b200.build [--force] [--verbose] [--debug]

``--debug`` builds ``liba2sf_debug.so`` from the same sources with ``-DA2SF_DEBUG``: every index
that addresses memory inside a kernel is range-checked and reported (``a2sf_debug_violations``)
instead of used.  Select it at run time with ``A2SF_LIBRARY=debug`` (see ``binding.py``).
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
OBJ_DIR = PKG / "_build"
LIB_PATH = PKG / "liba2sf.so"
DEBUG_OBJ_DIR = PKG / "_build_debug"
DEBUG_LIB_PATH = PKG / "liba2sf_debug.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (cand == "nvcc" or Path(cand).exists()):
            return cand
    raise RuntimeError("nvcc not found")


def _sources():
    return sorted(CSRC.glob("*.cu"))


def _deps_mtime() -> float:
    files = list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h"))
    return max(f.stat().st_mtime for f in files)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> Path:
    """Compile every ``csrc/*.cu`` and link the shared library (the bounds-checked one with
    ``debug``).  Returns its path."""
    obj_dir, lib_path = (DEBUG_OBJ_DIR, DEBUG_LIB_PATH) if debug else (OBJ_DIR, LIB_PATH)
    extra = ["-DA2SF_DEBUG"] if debug else []
    obj_dir.mkdir(exist_ok=True)
    nvcc = _nvcc()
    hdr_m = _deps_mtime()
    jobs = []
    for src in _sources():
        obj = obj_dir / (src.stem + ".o")
        if force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hdr_m):
            cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", str(INCLUDE), "-c", str(src), "-o", str(obj)]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed: {' '.join(cmd)}\n{r.stdout}\n{r.stderr}")
        return r.stderr

    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as ex:
        for log in ex.map(run, jobs):
            if verbose and log:
                print(log, file=sys.stderr)
    objs = [obj_dir / (s.stem + ".o") for s in _sources()]
    if force or jobs or not lib_path.exists():
        tmp = lib_path.with_suffix(f".tmp{os.getpid()}.so")
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
               "-o", str(tmp), *map(str, objs), "-cudart", "static"]
        run(cmd)
        os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
