"""Build ``libnsp.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

``python -m paper_2609_22755_b200.build`` compiles every ``csrc/*.cu`` (and the host-only ``csrc/*.cpp``) to an object file (in parallel) and links
them into ``paper_2609_22755_b200/libnsp.so`` with the CUDA runtime linked statically, so the library loads on a
machine without a GPU driver (the driver entry point it needs is resolved at run time).
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libnsp.so"
LIB_CHECKED = PKG / "libnsp_checked.so"  # the same sources with -DNSP_CHECKED: index checks inside the kernels
OBJ_DIR = PKG / "build"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
    "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and Path(cand).exists():
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(Path(d).stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    """Build libnsp.so, or with checked=True libnsp_checked.so (kernels verify every index they compute; for tests)."""
    nvcc = _nvcc()
    lib, tag, extra = (LIB_CHECKED, "_checked", ["-DNSP_CHECKED"]) if checked else (LIB, "", [])
    sources = sorted(CSRC.glob("*.cu")) + sorted(CSRC.glob("*.cpp"))  # the planner is host-only C++
    headers = sorted(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "nsp.h"]
    OBJ_DIR.mkdir(exist_ok=True)

    def compile_one(src: Path):
        obj = OBJ_DIR / (src.stem + tag + ".o")
        if force or _stale(obj, [src, *headers]):
            cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", str(src), "-o", str(obj)]
            r = subprocess.run(cmd, capture_output=True, text=True)
            (OBJ_DIR / (src.stem + tag + ".ptxas.log")).write_text(r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed for {src.name}:\n{r.stdout}\n{r.stderr}")
            if verbose:
                print(r.stderr, file=sys.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(sources))) as ex:
        objs = list(ex.map(compile_one, sources))
    if force or _stale(lib, objs):
        tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static",
               *map(str, objs), "-o", str(tmp)]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, checked=True))
