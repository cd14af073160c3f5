"""Builds the C-ABI CUDA library in-tree: ``python -m paper_2011_09398_b200.build``.

nvcc cross-compiles for sm_100a without a GPU present.  Every ``csrc/*.cu`` is compiled to an
object file (in parallel, only when it or a header changed) and the objects are linked into
``liblce_b200.so`` next to this file, which is what the binding loads.  ``csrc/probe/*.cu`` (pipe
micro-benchmarks used by bench.py only) goes into a library of its own, ``liblce_probe.so``.
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
OBJ = PKG / "build"
LIB = PKG / "liblce_b200.so"
PROBE_LIB = PKG / "liblce_probe.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(CSRC.glob("*.cu"))


def probe_sources():
    return sorted((CSRC / "probe").glob("*.cu"))


def _headers_mtime() -> float:
    deps = list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))
    return max(d.stat().st_mtime for d in deps)


def is_stale() -> bool:
    if not LIB.exists() or not PROBE_LIB.exists():
        return True
    t = min(LIB.stat().st_mtime, PROBE_LIB.stat().st_mtime)
    return any(s.stat().st_mtime > t for s in sources() + probe_sources()) or _headers_mtime() > t


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    OBJ.mkdir(exist_ok=True)
    hdr = _headers_mtime()
    jobs = []
    for src in sources() + probe_sources():
        obj = OBJ / (src.stem + ".o")
        if force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hdr):
            cmd = [nvcc, *NVCC_FLAGS, f"-I{INCLUDE}", f"-I{CSRC}", "-c", "-o", str(obj), str(src)]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    if verbose:
        for cmd in jobs:
            print(" ".join(cmd), file=sys.stderr)
    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        for res in pool.map(lambda c: subprocess.run(c, capture_output=not verbose, text=True), jobs):
            if res.returncode != 0:
                sys.stderr.write((res.stdout or "") + (res.stderr or ""))
                raise subprocess.CalledProcessError(res.returncode, res.args)
    stale = {p.stem for p in OBJ.glob("*.o")} - {s.stem for s in sources() + probe_sources()}
    for name in stale:  # objects of sources that no longer exist
        (OBJ / (name + ".o")).unlink()
    for lib, srcs in ((LIB, sources()), (PROBE_LIB, probe_sources())):
        tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
        objs = [str(OBJ / (s.stem + ".o")) for s in srcs]
        subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp), *objs], check=True)
        os.replace(tmp, lib)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
