"""Build libfosgd.so in-tree with nvcc for sm_100a (``python -m paper_2405_11095_b200.build``)."""
from __future__ import annotations

import concurrent.futures as cf
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
SO = os.path.join(HERE, "libfosgd.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]
ROW_TILES = (10, 11, 12, 13, 14, 15)


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _units():
    units = [("api.cu", "api.o", []), ("col_kernels.cu", "col_kernels.o", []),
             ("small_kernels.cu", "small_kernels.o", []), ("noalloc.cu", "noalloc.o", []), ("amplitudes.cu", "amplitudes.o", []),
             ("probe.cu", "probe.o", []), ("tc_kernels.cu", "tc_kernels.o", []),
             ("fused_encode.cu", "fused_encode.o", []), ("tc_row_kernels.cu", "tc_row_kernels.o", [])]
    units += [("row_inst.cu", f"row_{t}.o", [f"-DFOSGD_ROW_T={t}"]) for t in ROW_TILES]
    return units


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths.append(os.path.join(HERE, "..", "include", "fosgd.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(SO) and os.path.getmtime(SO) >= _newest_source():
        return SO
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(unit):
        src, obj, defs = unit
        cmd = [nvcc, *NVCC_FLAGS, *extra, *defs, "-c", os.path.join(CSRC, src), "-o", os.path.join(OBJ, obj)]
        r = subprocess.run(cmd, capture_output=True, text=True)
        return unit, r

    with cf.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 4)) as ex:
        for unit, r in ex.map(compile_one, _units()):
            if verbose or r.returncode != 0:
                sys.stderr.write(f"== {unit[1]}\n{r.stdout}{r.stderr}\n")
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed on {unit[0]} {unit[2]}")
    objs = [os.path.join(OBJ, u[1]) for u in _units()]
    tmp = SO + f".tmp{os.getpid()}"
    subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a",
                    "-cudart", "static"], check=True)
    os.replace(tmp, SO)
    return SO


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
