"""In-tree build of the C-ABI library ``libomni.so`` with nvcc for sm_100a."""
from __future__ import annotations

import fcntl
import hashlib
import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libomni.so"
SOURCES = [CSRC / "omni.cu", CSRC / "register_dispatch.cu", CSRC / "bulk_dispatch.cu", CSRC / "device_controller.cu", CSRC / "noalloc.cu",
           CSRC / "controller.cpp", CSRC / "shard.cpp"]
HEADERS = [CSRC / "kernels.cuh", CSRC / "tma_kernels.cuh", CSRC / "dispatch.h", CSRC / "controller.h",
           CSRC / "device_controller.h", PKG.parent / "include" / "omni.h"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC,-ffp-contract=off",
    "-shared",
]


STAMP = PKG / "libomni.so.sources"   # hash of the sources the library was built from


def source_hash() -> str:
    h = hashlib.sha256()
    for p in SOURCES + HEADERS:
        h.update(p.name.encode())
        h.update(p.read_bytes())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def stale() -> bool:
    """True when there is no library or it was built from other sources (content, not mtime:
    copying a tree does not keep modification times)."""
    if not LIB.exists() or not STAMP.exists():
        return True
    return STAMP.read_text().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every source to an object (in parallel), then link the shared library.  Safe to
    call from several processes at once (one builds, the others wait on a lock file)."""
    if not (force or stale()):
        return LIB
    lock = open(PKG / ".build.lock", "w")
    fcntl.flock(lock, fcntl.LOCK_EX)
    try:
        if not force and not stale():     # another process built it while we waited
            return LIB
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        objdir = PKG / "_build"
        objdir.mkdir(exist_ok=True)
        compile_flags = [f for f in NVCC_FLAGS if f != "-shared"] + (["-Xptxas", "-v"] if verbose else [])
        jobs = []
        for src in SOURCES:
            obj = objdir / (src.stem + f".{os.getpid()}.o")
            jobs.append((obj, subprocess.Popen([nvcc, *compile_flags, "-c", "-o", str(obj), str(src)])))
        failed = [str(o) for o, p in jobs if p.wait() != 0]
        if failed:
            raise RuntimeError(f"nvcc failed for {failed}")
        tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", str(tmp),
                        *[str(o) for o, _ in jobs]], check=True)
        os.replace(tmp, LIB)
        STAMP.write_text(source_hash() + "\n")
        for o, _ in jobs:
            o.unlink(missing_ok=True)
        return LIB
    finally:
        fcntl.flock(lock, fcntl.LOCK_UN)
        lock.close()


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
