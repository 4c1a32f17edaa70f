"""Compile the CUDA library in-tree: ``paper_2601_16536_b200/libw4a16.so`` (sm_100a only)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libw4a16.so")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(f) <= t for f in _deps())


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu of csrc/ to an object (in parallel) and link them into the shared library."""
    if not force and up_to_date():
        return LIB
    import concurrent.futures
    import tempfile
    flags = ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    with tempfile.TemporaryDirectory(prefix="w4a16_build_") as tmpdir:
        def compile_one(src):
            obj = os.path.join(tmpdir, os.path.basename(src)[:-3] + ".o")
            out = subprocess.run([_nvcc()] + flags + ["-c", src, "-o", obj], capture_output=True, text=True)
            return src, obj, out
        objs = []
        with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(sources()), os.cpu_count() or 1))) as ex:
            for src, obj, out in ex.map(compile_one, sources()):
                if verbose or out.returncode != 0:
                    sys.stderr.write(out.stdout + out.stderr)
                if out.returncode != 0:
                    raise RuntimeError("nvcc failed on %s" % src)
                objs.append(obj)
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([_nvcc(), "-shared", "-o", tmp] + objs)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
