"""Build libscissorhands.so in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB_DIR = os.path.join(PKG, "lib")
LIB = os.path.join(LIB_DIR, "libscissorhands.so")
LIB_DEBUG_BOUNDS = os.path.join(LIB_DIR, "libscissorhands_bounds.so")
INCLUDE = os.path.join(ROOT, "include")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: cannot build libscissorhands.so")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    mt = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.inl")) \
        + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(f) > mt for f in deps)


def build(force: bool = False, verbose: bool = False, out: str = LIB, debug_bounds: bool = False) -> str:
    """Compile every .cu under csrc/ (one nvcc process per file, in parallel) and link them into one shared
    library.  Returns its path.  ``debug_bounds``: the bounds-checked build (-DSH_DEBUG_BOUNDS: every index a
    kernel derives from workspace state is range-checked and a violation is reported through the device error
    word instead of being dereferenced), written to lib/libscissorhands_bounds.so."""
    if debug_bounds and out == LIB:
        out = LIB_DEBUG_BOUNDS
    if not force and os.path.exists(out) and not stale(out):
        return out
    os.makedirs(os.path.dirname(out), exist_ok=True)
    obj_dir = os.path.join(os.path.dirname(out), f"obj.{os.getpid()}")
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", INCLUDE, "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    if debug_bounds:
        flags += ["-DSH_DEBUG_BOUNDS"]
    try:
        jobs = []
        for src in sources():
            obj = os.path.join(obj_dir, os.path.basename(src) + ".o")
            jobs.append((src, obj, subprocess.Popen([nvcc, *flags, "-c", src, "-o", obj], stdout=subprocess.PIPE,
                                                    stderr=subprocess.STDOUT, text=True)))
        log = []
        for src, obj, proc in jobs:
            text, _ = proc.communicate()
            log.append(text)
            if proc.returncode != 0:
                for _s, _o, other in jobs:
                    if other.poll() is None:
                        other.kill()
                raise RuntimeError(f"nvcc failed on {os.path.basename(src)}:\n{text}")
        tmp = out + f".{os.getpid()}.tmp"
        res = subprocess.run([nvcc, "-shared", "-o", tmp, *[obj for _s, obj, _p in jobs]], capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
        if verbose:
            print("".join(log))
        os.replace(tmp, out)
    finally:
        shutil.rmtree(obj_dir, ignore_errors=True)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
