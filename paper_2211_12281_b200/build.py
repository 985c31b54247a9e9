"""Builds libkge.so (sm_100a) in-tree with nvcc.  No GPU is needed to compile.

Every source is compiled to an object of its own (in parallel, only when it or a header has
changed) under ``_build/`` and the objects are linked into ``libkge.so`` beside this file.
"""
from __future__ import annotations

import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libkge.so"
OBJ = PKG / "_build"
SOURCES = ["kge_api.cu", "kge_sample.cu", "kge_train.cu", "kge_tc.cu", "kge_update.cu", "kge_infer.cu",
           "kge_graph.cu", "kge_ensemble.cu", "kge_bench.cu", "kge_transh.cu", "kge_encoder.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(cand).exists():
        raise RuntimeError("nvcc not found")
    return cand


def _headers_mtime() -> float:
    heads = [p for p in CSRC.iterdir() if p.suffix in (".cuh", ".h")] + [PKG.parent / "include" / "kge.h"]
    return max(p.stat().st_mtime for p in heads)


def needs_build() -> bool:
    if not LIB.exists():
        return True
    newest = max(max(p.stat().st_mtime for p in CSRC.iterdir()), _headers_mtime())
    return newest > LIB.stat().st_mtime


def _compile(src: Path, obj: Path, verbose: bool) -> str:
    cmd = [nvcc_path(), "-O3", "-std=c++17", *ARCH, "-lineinfo", "-Xcompiler", "-fPIC",
           "-Xptxas", "-v" if verbose else "-O3", "-c", str(src), "-o", str(obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src.name}:\n" + res.stdout + res.stderr)
    return res.stdout + res.stderr


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    OBJ.mkdir(exist_ok=True)
    hm = _headers_mtime()
    jobs = []
    for name in SOURCES:
        src, obj = CSRC / name, OBJ / (name + ".o")
        stale = force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hm)
        if stale:
            jobs.append((src, obj))
    with ThreadPoolExecutor(max_workers=8) as pool:
        logs = list(pool.map(lambda j: _compile(j[0], j[1], verbose), jobs))
    if verbose:
        print("".join(logs), file=sys.stderr)
    link = [nvcc_path(), *ARCH, "-shared", "-Xcompiler", "-fPIC", *[str(OBJ / (n + ".o")) for n in SOURCES], "-o", str(LIB)]
    res = subprocess.run(link, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    build(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
