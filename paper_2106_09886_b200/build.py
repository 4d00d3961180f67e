"""Build libqnn.so from csrc/*.cu with nvcc for sm_100a (no torch involved).

    python -m paper_2106_09886_b200.build [--force]
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libqnn.so"
STAMP = PKG / "libqnn.so.digest"

COMPILE_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",            # no silent contraction: every fused multiply-add is written explicitly
    "-Xcompiler", "-fPIC", "-Xcompiler", "-O2",
]
LINK_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC"]


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def _digest() -> str:
    """Content digest of everything the library is built from (file times do not survive copies of the tree)."""
    h = hashlib.sha256()
    h.update(" ".join(COMPILE_FLAGS + LINK_FLAGS).encode())
    for path in sources() + sorted(CSRC.glob("*.cuh")) + sorted(INCLUDE.glob("*.h")):
        h.update(path.name.encode())
        h.update(path.read_bytes())
    return h.hexdigest()


def needs_build() -> bool:
    return not LIB.exists() or not STAMP.exists() or STAMP.read_text().strip() != _digest()


def _compile(nvcc: str, src: Path, obj: Path, verbose: bool) -> str:
    cmd = [nvcc, *COMPILE_FLAGS, f"-I{INCLUDE}", f"-I{CSRC}", "-c", "-o", str(obj), str(src)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src.name}:\n{r.stdout}\n{r.stderr}")
    return r.stderr


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every csrc/*.cu to an object file (in parallel) and link them into libqnn.so."""
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = PKG / "_build"
    objdir.mkdir(exist_ok=True)
    srcs = sources()
    objs = [objdir / (s.stem + ".o") for s in srcs]
    workers = max(1, min(len(srcs), os.cpu_count() or 1))
    with ThreadPoolExecutor(max_workers=workers) as pool:
        logs = list(pool.map(lambda so: _compile(nvcc, so[0], so[1], verbose), zip(srcs, objs)))
    if verbose:
        print("".join(logs), file=sys.stderr)
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.check_call([nvcc, *LINK_FLAGS, "-o", str(tmp), *map(str, objs)])
    os.replace(tmp, LIB)
    STAMP.write_text(_digest() + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
