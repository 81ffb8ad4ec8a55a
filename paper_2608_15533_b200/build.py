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
    "--threads", "0",   # the translation units under csrc/ compile side by side
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
    for path in sorted(list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h"))):
        h.update(path.name.encode())
        h.update(path.read_bytes())
    h.update(" ".join([*NVCC_FLAGS, *extra]).encode())
    return h.hexdigest()[:12]


# A second build of the same sources for one test: waits inside the kernels give up after 5 ms instead
# of 2 s, and the decode kernel accepts the index of one unit whose first chunk it never requests, so
# that the give-up path of the bounded waits can be exercised without hanging or faulting anything.
TEST_HOOKS_LIB = PKG / "libdeltalog_testhooks.so"
TEST_HOOKS_FLAGS = ["-DDELTALOG_WAIT_LIMIT_NS=5000000ull", "-DDELTALOG_TEST_HOOKS=1"]


def _stale(lib: Path) -> bool:
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h")) + [Path(__file__)]
    return any(d.stat().st_mtime > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, lib: Path = LIB, extra=None) -> Path:
    """Build ``libdeltalog.so`` next to this file if it is missing or older than its sources (``lib`` /
    ``extra``: another output file with additional compiler switches)."""
    if not force and not _stale(lib):
        return lib
    tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
    extra = extra_flags() + list(extra or [])
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, f'-DDELTALOG_BUILD_ID="{source_id(extra)}"', f"-I{INCLUDE}", f"-I{CSRC}",
           *map(str, sources()), "-o", str(tmp)]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        tmp.unlink(missing_ok=True)
        raise RuntimeError(f"nvcc failed ({proc.returncode}): {' '.join(cmd)}")
    if lib == LIB:
        (PKG / "ptxas_info.txt").write_text(proc.stdout + proc.stderr)
    os.replace(tmp, lib)
    return lib


def build_test_hooks_library(force: bool = False) -> Path:
    return build_library(force=force, lib=TEST_HOOKS_LIB, extra=TEST_HOOKS_FLAGS)


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True))
    if "--test-hooks" in sys.argv:
        print(build_test_hooks_library(force="--force" in sys.argv))
