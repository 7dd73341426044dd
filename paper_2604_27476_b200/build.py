"""Build libedgefm.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libedgefm.so"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def sources():
    return sorted(CSRC.glob("*.cu"))


STAMP = PKG / "libedgefm.so.srchash"


def source_hash() -> str:
    """Hash of everything the library is built from (content, not time stamps: a copied tree keeps its build)."""
    import hashlib
    h = hashlib.sha256()
    deps = sorted(list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h"))) + [PKG.parent / "include" / "edgefm.h"]
    for p in deps:
        h.update(p.name.encode())
        h.update(p.read_bytes())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def needs_build() -> bool:
    if not LIB.exists() or not STAMP.exists():
        return True
    return STAMP.read_text().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math") and f != "-shared"]
    objdir = PKG / "build"
    objdir.mkdir(exist_ok=True)
    # one object per translation unit, compiled in parallel (the kernel variants dominate the build time)
    from concurrent.futures import ThreadPoolExecutor

    def compile_one(src: Path) -> Path:
        obj = objdir / (src.stem + f".{os.getpid()}.o")
        subprocess.check_call([nvcc, *flags, *(["-Xptxas", "-v"] if verbose else []), "-c", "-o", str(obj), str(src)])
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    subprocess.check_call([nvcc, "-shared", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a", "-o", str(tmp),
                           *map(str, objs)])
    for o in objs:
        o.unlink(missing_ok=True)
    os.replace(tmp, LIB)
    STAMP.write_text(source_hash() + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
