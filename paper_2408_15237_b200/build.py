"""Builds ``libmamba_spec.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Run as ``python -m paper_2408_15237_b200.build``; ``build_library()`` is what the
repository's build entry point calls.  The library is rebuilt only when a source
is newer than it.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libmamba_spec.so"
SOURCES = ["mamba_spec.cu", "verify_generic.cu", "verify_stream.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return exe


def _stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "mamba_spec.h"]
    return any(d.stat().st_mtime > lib.stat().st_mtime for d in deps)


# Test-only build: the same sources with waits that give up after about a millisecond and a barrier that can
# never complete, so that the kernel's give-up path runs (every copy still lands; see tests/test_gpu_waits.py).
WAIT_TEST_LIB = PKG / "_build" / "libmamba_spec_waittest.so"
WAIT_TEST_DEFINES = ["-DMSPEC_WAIT_LIMIT_CYCLES=2000000ll", "-DMSPEC_TEST_RAW_NEVER_FULL=1"]


def build_wait_test_library(force: bool = False) -> Path:
    return build_library(force=force, defines=WAIT_TEST_DEFINES, out=WAIT_TEST_LIB, tag="waittest")


def build_library(force: bool = False, verbose: bool = False, defines=(), out: Path = LIB, tag: str = "") -> Path:
    if not force and not _stale(out):
        return out
    objs = []
    out_dir = PKG / "_build"
    out_dir.mkdir(exist_ok=True)
    extra = (["-Xptxas", "-v"] if verbose else []) + list(defines)
    procs = []
    for src in SOURCES:
        obj = out_dir / (src + (f".{tag}" if tag else "") + ".o")
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", str(CSRC / src), "-o", str(obj)]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, pr in procs:
        log, _ = pr.communicate()
        if verbose or pr.returncode:
            sys.stderr.write(log)
        if pr.returncode:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = out.parent / f".{out.stem}.{os.getpid()}.so"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", str(tmp), *map(str, objs),
           "-lcudart"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
