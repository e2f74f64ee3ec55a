"""Build the CUDA library in-tree: ``python -m paper_1804_10727_b200.build``.

Compiles every ``csrc/*.cu`` for sm_100a with nvcc and links ``libidf.so`` next
to this file (cross-compiles without a GPU).
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libidf.so"
BOUNDS_LIB = HERE / "libidf_bounds.so"      # the same sources with every index range-checked (-DIDF_BOUNDS)
INCLUDE = HERE.parent / "include"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
]


def sources():
    return sorted(CSRC.glob("*.cu"))


def _stale() -> bool:
    if not LIB.exists() or not BOUNDS_LIB.exists():
        return True
    t = min(LIB.stat().st_mtime, BOUNDS_LIB.stat().st_mtime)
    deps = list(CSRC.glob("*")) + list(INCLUDE.glob("*.h"))
    return any(p.stat().st_mtime > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = {LIB: [], BOUNDS_LIB: []}
    procs = []
    for lib, extra, suffix in ((LIB, [], ".o"), (BOUNDS_LIB, ["-DIDF_BOUNDS"], ".bounds.o")):
        for src in sources():
            obj = src.with_suffix(suffix)
            cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", str(INCLUDE), "-c", str(src), "-o", str(obj)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
            objs[lib].append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if out.strip() and (verbose or p.returncode != 0):
            print(f"--- {src.name}\n{out}", file=sys.stderr)
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    for lib, lib_objs in objs.items():
        tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run([nvcc, "-shared", "-o", str(tmp), *map(str, lib_objs)], check=True)
        os.replace(tmp, lib)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
