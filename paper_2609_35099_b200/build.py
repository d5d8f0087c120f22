"""Ahead-of-time build of libe3j.so (sm_100a only).

    python -m paper_2609_35099_b200.build [--force] [--verbose] [--signatures extra.json] [--out lib.so]

Every translation unit under csrc/ (and the generated ones under csrc/fast/) is
compiled with nvcc for compute_100a / sm_100a and linked into
paper_2609_35099_b200/libe3j.so.  nvcc cross-compiles without a GPU.  Object files
and the ptxas resource report (registers, spills, shared memory) go to csrc/build/.

Signatures beyond the committed list: --signatures names a JSON list of entries like
    {"name": "w96_l2", "irreps_in": "96x0e+96x1o", "sh_lmax": 2, "irreps_out": null, "out_lmax": 2}
(tile parameters optional: the generator derives what is missing from shared-memory and register fits).  Their
kernels are generated into csrc/build/overlay/ (git-ignored) with the library that the normal build produced,
compiled, and linked with everything else into --out (default: libe3j.so itself).  A plan with such a signature
then selects the generated kernels like any committed one; without the overlay it runs on the table-driven ones.
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


def _link(objs, out: Path) -> None:
    tmp = out.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp),
           *map(str, objs), "-cudart", "static"]
    subprocess.check_call(cmd)
    os.replace(tmp, out)


def build(force: bool = False, verbose: bool = False) -> Path:
    BUILD.mkdir(parents=True, exist_ok=True)
    digest = _deps_digest()
    srcs = sources()
    with cf.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(lambda s: _compile(s, digest, force, verbose), srcs))
    newest = max(o.stat().st_mtime for o in objs)
    if force or not OUT.exists() or OUT.stat().st_mtime < newest:
        _link(objs, OUT)
    return OUT


def build_overlay(signatures: Path, out: Path | None = None, verbose: bool = False) -> Path:
    """The library plus generated kernels for the signatures listed in `signatures` (see the module docstring)."""
    import importlib.util
    import json
    build()   # the generator asks the built library for the coefficient records
    spec = importlib.util.spec_from_file_location("e3j_gen_fast", CSRC / "gen_fast.py")
    gen = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(gen)
    extra = json.loads(Path(signatures).read_text())
    files = gen.generate(extra)
    over = BUILD / "overlay"
    over.mkdir(parents=True, exist_ok=True)
    names = {s["name"] for s in extra}
    new_srcs = []
    for fname, text in files.items():
        if fname == "registry_entries.inc" or fname[len("sig_"):-len(".cu")] in names:
            (over / fname).write_text(text)
            if fname.endswith(".cu"):
                new_srcs.append(over / fname)
    digest = _deps_digest()
    flags = NVCC_FLAGS + ["-I", str(CSRC / "fast"), "-I", str(CSRC)]
    objs = []
    for src in sources():
        if src.name == "fast_registry.cu":   # recompiled against the overlay's entry list
            obj = over / "fast_registry.o"
            cmd = ["nvcc", *flags, f'-DE3J_REGISTRY_INC="{over / "registry_entries.inc"}"', "-x", "cu", "-c", str(src), "-o", str(obj)]
            subprocess.check_call(cmd)
            objs.append(obj)
        else:
            objs.append(_compile(src, digest, False, verbose))
    for src in new_srcs:
        obj = over / (src.stem + ".o")
        res = subprocess.run(["nvcc", *flags, "-x", "cu", "-c", str(src), "-o", str(obj)], capture_output=True, text=True)
        (over / (src.stem + ".ptxas.log")).write_text(res.stderr)
        if res.returncode != 0:
            sys.stderr.write(res.stderr)
            raise RuntimeError(f"nvcc failed on {src.name}")
        objs.append(obj)
    out = Path(out) if out else OUT
    _link(objs, out)
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    ap.add_argument("--signatures", help="JSON list of extra signatures to generate kernels for (overlay build)")
    ap.add_argument("--out", help="where the overlay build writes its library (default: libe3j.so)")
    a = ap.parse_args()
    print(build_overlay(a.signatures, a.out, a.verbose) if a.signatures else build(a.force, a.verbose))
