"""Compile the CUDA sources under ``csrc/`` into ``libdeltalog.so`` (sm_100a only, in-tree)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libdeltalog.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "--shared", "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and Path(cand).exists():
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def sources():
    return sorted(CSRC.glob("*.cu"))


def extra_flags():
    """Extra compiler switches for experiments (``DELTALOG_NVCC_EXTRA="-D..."``)."""
    return os.environ.get("DELTALOG_NVCC_EXTRA", "").split()


def source_id(extra=()) -> str:
    """Twelve hex digits identifying what the library is built from: every file under ``csrc/``, the
    header and the compiler switches.  It is compiled into the library (``deltalog_build_id``), and
    profiler figures kept beside the code carry it, so a figure taken from another build is recognised."""
    import hashlib

    h = hashlib.sha256()
    for path in sorted(list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))):
        h.update(path.name.encode())
        h.update(path.read_bytes())
    h.update(" ".join([*NVCC_FLAGS, *extra]).encode())
    return h.hexdigest()[:12]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h")) + [Path(__file__)]
    return any(d.stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> Path:
    """Build ``libdeltalog.so`` next to this file if it is missing or older than its sources."""
    if not force and not _stale():
        return LIB
    tmp = LIB.with_suffix(f".so.tmp{os.getpid()}")
    extra = extra_flags()
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, f'-DDELTALOG_BUILD_ID="{source_id(extra)}"', f"-I{INCLUDE}", f"-I{CSRC}",
           *map(str, sources()), "-o", str(tmp)]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        tmp.unlink(missing_ok=True)
        raise RuntimeError(f"nvcc failed ({proc.returncode}): {' '.join(cmd)}")
    (PKG / "ptxas_info.txt").write_text(proc.stdout + proc.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True))
