"""Ahead-of-time build of libe3j.so (sm_100a only).

    python -m paper_2609_35099_b200.build [--force] [--verbose]

Every translation unit under csrc/ (and the generated ones under csrc/fast/) is
compiled with nvcc for compute_100a / sm_100a and linked into
paper_2609_35099_b200/libe3j.so.  nvcc cross-compiles without a GPU.  Object files
and the ptxas resource report (registers, spills, shared memory) go to csrc/build/.
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import hashlib
import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
OUT = PKG / "libe3j.so"
BUILD = CSRC / "build"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v", "--expt-relaxed-constexpr",
] + os.environ.get("E3J_NVCC_EXTRA", "").split()   # e.g. -DE3J_RADIAL_PROF (role cycle counters of fast_radial.cuh)


def sources() -> list[Path]:
    srcs = sorted(CSRC.glob("*.cpp")) + sorted(CSRC.glob("*.cu")) + sorted((CSRC / "fast").glob("*.cu"))
    return srcs


def _deps_digest() -> str:
    h = hashlib.sha256()
    for p in sorted(list(CSRC.glob("*.hpp")) + list(CSRC.glob("*.cuh")) + list((CSRC / "fast").glob("*.inc"))
                    + list((CSRC / "fast").glob("*.cuh")) + [PKG.parent / "include" / "e3j.h"]):
        h.update(p.read_bytes())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()[:16]


def _compile(src: Path, digest: str, force: bool, verbose: bool) -> Path:
    obj = BUILD / (src.stem + ".o")
    stamp = BUILD / (src.stem + ".stamp")
    key = hashlib.sha256(src.read_bytes()).hexdigest()[:16] + digest
    if not force and obj.exists() and stamp.exists() and stamp.read_text() == key:
        return obj
    cmd = ["nvcc", *NVCC_FLAGS, "-x", "cu", "-c", str(src), "-o", str(obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    (BUILD / (src.stem + ".ptxas.log")).write_text(res.stderr)
    if res.returncode != 0:
        sys.stderr.write(res.stderr)
        raise RuntimeError(f"nvcc failed on {src.name}")
    if verbose:
        sys.stderr.write(res.stderr)
    stamp.write_text(key)
    return obj


def build(force: bool = False, verbose: bool = False) -> Path:
    BUILD.mkdir(parents=True, exist_ok=True)
    digest = _deps_digest()
    srcs = sources()
    with cf.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(lambda s: _compile(s, digest, force, verbose), srcs))
    newest = max(o.stat().st_mtime for o in objs)
    if force or not OUT.exists() or OUT.stat().st_mtime < newest:
        tmp = OUT.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp),
               *map(str, objs), "-cudart", "static"]
        subprocess.check_call(cmd)
        os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    a = ap.parse_args()
    print(build(a.force, a.verbose))
