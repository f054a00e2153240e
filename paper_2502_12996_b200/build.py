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
OUTER_M = [0, 1, 2, 3, 4, 8, 16, 1000, 1002, 1003, 1004]   # translation units: replica counts with kernels of their own, the
                                                 # warp-split forms (1000, 1002) and the first-steps form (0)
OBJ = PKG / "_obj"

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-fmad=false",                       # no FMA contraction: one rounding per operation
    "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
] + os.environ.get("DILOCO_EXTRA_NVCC_FLAGS", "").split()


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "diloco.h", Path(__file__)]
    return any(d.stat().st_mtime > t for d in deps)


def _compile(nvcc: str, src: Path, obj: Path, defines) -> str:
    cmd = [nvcc] + NVCC_FLAGS + [f"-D{d}" for d in defines] + ["-c", str(src), "-o", str(obj)]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if res.returncode != 0:
        print(res.stdout)
        raise subprocess.CalledProcessError(res.returncode, cmd)
    return res.stdout


def build_library(force: bool = False, verbose: bool = False) -> Path:
    """Compile the host/ABI unit and one unit per replica count side by side, then link."""
    if not force and not _stale() and REPORT.exists():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    OBJ.mkdir(exist_ok=True)
    jobs = [(CSRC / "diloco_api.cu", OBJ / "diloco_api.o", []),
            (CSRC / "diloco_utilization.cu", OBJ / "diloco_utilization.o", [])]
    jobs += [(CSRC / "diloco_outer_m.cu", OBJ / f"diloco_outer_m{m}.o", [f"DILOCO_M={m}"]) for m in OUTER_M]
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
        logs = list(pool.map(lambda j: _compile(nvcc, *j), jobs))
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    link = [nvcc, "-shared", "--cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp)] \
        + [str(j[1]) for j in jobs]
    subprocess.check_call(link)
    report = "\n".join(logs)
    if verbose:
        print(report)
    REPORT.write_text(report)
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
