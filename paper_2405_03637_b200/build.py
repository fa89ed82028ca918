"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2405_03637_b200.build [--force] [--verbose] [--define NAME[=VALUE]]... [--out PATH]

--define adds a preprocessor definition (the geometry constants COLLAGE_PIPE_* / COLLAGE_FP32_*, or
COLLAGE_DATA_MOVEMENT_ONLY, which compiles the arithmetic out of the step kernel to measure what the
copy pipeline alone sustains); such a build goes to --out, never over the in-tree library, and is
loaded only on request: `binding.load(path)`, which `bench.py --lib PATH` calls.

The exactness of the error-free transforms depends on the flags below: no FMA contraction,
no flush-to-zero, IEEE division and square root, never --use_fast_math.
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libcollage_b200.so"
SOURCES = ["collage_step.cu", "collage_primitives.cu", "collage_edq_static.cu", "collage_fp32_master.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
    "--split-compile", "0", "-t", "0",      # compile the many kernel instantiations on all host cores
]


def _newest_source_mtime() -> float:
    files = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [HERE.parent / "include" / "collage.h", Path(__file__)]
    return max(f.stat().st_mtime for f in files)


def build(force: bool = False, verbose: bool = False, defines: tuple = (), out: Path | None = None) -> Path:
    if defines and out is None:
        raise ValueError("a build with extra definitions needs its own output path")
    lib = Path(out) if out is not None else LIB
    if out is None and not force and LIB.exists() and LIB.stat().st_mtime >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, *NVCC_FLAGS, *[f"-D{d}" for d in defines], *(["-Xptxas", "-v"] if verbose else []), "-o", str(tmp),
           *[str(CSRC / s) for s in SOURCES]]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode:
        raise RuntimeError("nvcc failed building the Collage CUDA library")
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    argv = sys.argv[1:]
    defs = tuple(argv[i + 1] for i, a in enumerate(argv) if a == "--define" and i + 1 < len(argv))
    outp = next((Path(argv[i + 1]) for i, a in enumerate(argv) if a == "--out" and i + 1 < len(argv)), None)
    print(build(force="--force" in argv, verbose="--verbose" in argv, defines=defs, out=outp))
