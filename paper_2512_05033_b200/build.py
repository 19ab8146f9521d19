"""Build libarb.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2512_05033_b200.build [--force] [--verbose] [--checks]

--checks builds libarb_checks.so instead: the same sources with -DARB_CHECKS (device-side range tests that raise
ARB_DEV_CHECK_FAILED and skip the access, guard zones around the buffers a context owns).  The binding loads it when
ARB_LIB_VARIANT=checks is set; it is for test runs, not for timing.
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
OBJ = HERE / "_build"
LIB = HERE / "libarb.so"
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
         "-Xcompiler", "-fPIC", "--use_fast_math"]


def _sources():
    return sorted(CSRC.glob("*.cu"))


def _stale(target: Path, deps) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False, checks: bool = False) -> Path:
    headers = list(CSRC.glob("*.cuh")) + [HERE.parent / "include" / "arb.h", Path(__file__)]
    OBJ = HERE / ("_build_checks" if checks else "_build")
    LIB = HERE / ("libarb_checks.so" if checks else "libarb.so")
    OBJ.mkdir(exist_ok=True)
    jobs = []
    for src in _sources():
        obj = OBJ / (src.stem + ".o")
        if force or _stale(obj, [src] + headers):
            cmd = [NVCC, *FLAGS, *(["-DARB_CHECKS"] if checks else []), "-c", str(src), "-o", str(obj)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for cmd, res in zip(jobs, ex.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs)):
                if verbose or res.returncode != 0:
                    sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
                if res.returncode != 0:
                    raise RuntimeError(f"nvcc failed on {cmd[-3]}")
    objs = [OBJ / (s.stem + ".o") for s in _sources()]
    if force or jobs or _stale(LIB, objs):
        tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call([NVCC, "-shared", "-Wno-deprecated-gpu-targets", "-o", str(tmp), *map(str, objs),
                               "-lcudart"])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checks="--checks" in sys.argv))
