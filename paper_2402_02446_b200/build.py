"""Build the CUDA library in-tree: nvcc (sm_100a) -> paper_2402_02446_b200/lib/liblqer.so."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OUT_DIR = os.path.join(HERE, "lib")
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(OUT_DIR, "liblqer.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def sources() -> list[str]:
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _stale(target: str, deps: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


LIB_DEBUG = os.path.join(OUT_DIR, "liblqer_dbg.so")


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compiles the library.  debug_bounds: the checked build (-DLQER_DEBUG_BOUNDS -> lib/liblqer_dbg.so), whose kernels
    check every global store and weight copy against its buffer's extent and report the first violation through the
    status word; the binding loads it when LQER_DEBUG_BOUNDS=1 is in the environment."""
    OBJ_DIR = os.path.join(HERE, "_build_dbg" if debug_bounds else "_build")
    LIB = LIB_DEBUG if debug_bounds else globals()["LIB"]
    NVCC_FLAGS = globals()["NVCC_FLAGS"] + (["-DLQER_DEBUG_BOUNDS"] if debug_bounds else [])
    os.makedirs(OUT_DIR, exist_ok=True)
    os.makedirs(OBJ_DIR, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(ROOT, "include", "lqer.h"))
    nvcc = _nvcc()
    jobs = []
    for src in sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        if force or _stale(obj, [src] + headers):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        r = subprocess.run([nvcc, *NVCC_FLAGS, "-c", src, "-o", obj], capture_output=True, text=True)
        return src, r

    with ThreadPoolExecutor(max_workers=8) as ex:
        for src, r in ex.map(compile_one, jobs):
            if verbose or r.returncode != 0:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed on {src}")
            with open(os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".ptxas.txt"), "w") as f:
                f.write(r.stderr)
    objs = [os.path.join(OBJ_DIR, os.path.basename(s)[:-3] + ".o") for s in sources()]
    if force or jobs or _stale(LIB, objs):
        r = subprocess.run([nvcc, "-shared", "-o", LIB, *objs], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return LIB


def build_all(force: bool = False, verbose: bool = False) -> list[str]:
    """The library and its checked build."""
    return [build(force, verbose), build(force, verbose, debug_bounds=True)]


if __name__ == "__main__":
    for path in build_all(force="--force" in sys.argv, verbose="-v" in sys.argv):
        print(path)
