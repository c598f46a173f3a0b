"""Build libtpq.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libtpq.so"

OBJ = PKG / "build"   # object files (git-ignored)

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC",
    # IEEE arithmetic everywhere: no fast-math; the kernels use explicit _rn intrinsics
    # wherever the rounding sequence is part of the result.
]
LINK_FLAGS = ["-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC"]


def sources():
    return sorted(CSRC.glob("*.cu"))


def _stale(target: Path, deps) -> bool:
    return (not target.exists()) or target.stat().st_mtime < max(d.stat().st_mtime for d in deps)


def needs_build() -> bool:
    return _stale(LIB, list(CSRC.glob("*")) + [INCLUDE / "tpq.h", Path(__file__)])


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every translation unit to an object file (only the stale ones unless ``force``), side by side,
    and link them into libtpq.so."""
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    OBJ.mkdir(exist_ok=True)
    headers = list(CSRC.glob("*.h")) + [INCLUDE / "tpq.h", Path(__file__)]
    jobs = []
    for src in sources():
        obj = OBJ / (src.stem + ".o")
        if force or _stale(obj, [src] + headers):
            cmd = [nvcc, *NVCC_FLAGS, "-c", f"-I{INCLUDE}", f"-I{CSRC}", "-o", str(obj), str(src)]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)))
    failed = []
    for src, proc in jobs:
        out, err = proc.communicate()
        if verbose:
            sys.stderr.write(err)
        if proc.returncode != 0:
            failed.append(f"{src.name}:\n{out}{err}")
    if failed:
        raise RuntimeError("nvcc failed:\n" + "\n".join(failed))
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    objs = [str(OBJ / (src.stem + ".o")) for src in sources()]
    res = subprocess.run([nvcc, *LINK_FLAGS, "-o", str(tmp), *objs], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
