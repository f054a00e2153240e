"""In-tree build of libdiloco.so with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libdiloco.so"
REPORT = PKG / "ptxas_report.txt"        # registers / spills of every kernel, written by each build
SOURCES = [CSRC / "diloco_api.cu"]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-fmad=false",                       # no FMA contraction: one rounding per operation
    "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "--cudart", "static", "-shared", "-Xcompiler", "-fPIC",
]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "diloco.h", Path(__file__)]
    return any(d.stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> Path:
    if not force and not _stale() and REPORT.exists():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc] + NVCC_FLAGS + ["-Xptxas", "-v", "-o", str(tmp)] + [str(s) for s in SOURCES]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout)
    if res.returncode != 0:
        raise subprocess.CalledProcessError(res.returncode, cmd)
    REPORT.write_text(res.stdout)
    os.replace(tmp, LIB)
    return LIB


def kernel_resources():
    """(mangled name, registers, spill-store bytes, stack bytes) of every kernel in the last build."""
    import re
    out = []
    for block in REPORT.read_text().split("Compiling entry function '")[1:]:
        name = block.split("'")[0]
        regs = int(re.search(r"Used (\d+) registers", block).group(1))
        spill = int(re.search(r"(\d+) bytes spill stores", block).group(1))
        stack = int(re.search(r"(\d+) bytes stack frame", block).group(1))
        out.append((name, regs, spill, stack))
    return out


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
