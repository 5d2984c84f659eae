"""Builds the CUDA library in-tree: csrc/*.cu -> libsbw.so next to this file (sm_100a only)."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

_HERE = Path(__file__).resolve().parent
CSRC = _HERE / "csrc"
INCLUDE = _HERE.parent / "include"
LIB = _HERE / "libsbw.so"
LIB_DEBUG = _HERE / "libsbw_debug.so"     # the bounds-flag build (-DSBW_DEBUG), used by one GPU test only

def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(exe).exists():
        raise RuntimeError("nvcc not found: the SBW CUDA library cannot be built")
    return exe


def sources() -> list[Path]:
    return sorted(CSRC.glob("*.cu"))


def is_stale(lib: Path | None = None) -> bool:
    lib = LIB if lib is None else lib
    if not lib.exists():
        return True
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))
    return lib.stat().st_mtime < max(p.stat().st_mtime for p in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> Path:
    """Compile every kernel for sm_100a and link libsbw.so.  Needs nvcc, not a GPU.  The sources
    are compiled to objects side by side (one nvcc per file), then linked.  debug=True builds the
    bounds-flag variant libsbw_debug.so instead (checked accesses that record failures in a device
    flag; relocatable device code because the flag is shared by all sources)."""
    target = LIB_DEBUG if debug else LIB
    if not force and not is_stale(target):
        return target
    import tempfile
    from concurrent.futures import ThreadPoolExecutor

    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", str(INCLUDE)]
    if verbose:
        flags += ["-Xptxas", "-v"]
    if debug:
        flags += ["-DSBW_DEBUG", "-rdc=true"]
    with tempfile.TemporaryDirectory(prefix="sbw_build_") as tmpdir:
        def compile_one(src: Path) -> str:
            obj = str(Path(tmpdir) / (src.stem + ".o"))
            subprocess.run([_nvcc(), *flags, "-c", str(src), "-o", obj], check=True)
            return obj

        srcs = sources()
        with ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 4)) as pool:
            objects = list(pool.map(compile_one, srcs))
        tmp = target.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "shared",
                        "-o", str(tmp), *objects], check=True)
        os.replace(tmp, target)
    return target


if __name__ == "__main__":
    import sys

    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
