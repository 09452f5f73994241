"""Builds libresps.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libresps.so")
SOURCES = ["api.cu", "scan.cu", "tree.cu", "attention.cu", "accept.cu", "sampled.cu", "controller.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _newer(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


WAIT_TEST_LIB = os.path.join(HERE, "libresps_waittest.so")


def build(force: bool = False, verbose: bool = False, wait_test: bool = False) -> str:
    """Builds the library.  wait_test=True builds the separate test library instead
    (-DRESPS_WAIT_TEST: millisecond wait limits and a switch that leaves out one copy); it is
    loaded by the bounded-wait test only, never by the binding."""
    nvcc = os.environ.get("NVCC", "nvcc")
    if wait_test:
        return _build_into(nvcc, os.path.join(OBJ, "waittest"), WAIT_TEST_LIB, ["-DRESPS_WAIT_TEST"], force, verbose)
    return _build_into(nvcc, OBJ, LIB, [], force, verbose)


def _build_into(nvcc, OBJ, LIB, extra_flags, force, verbose) -> str:
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(ROOT, "include", "resps.h"))
    jobs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src.replace(".cu", ".o"))
        if force or _newer(o, [s] + headers):
            cmd = [nvcc] + NVCC_FLAGS + extra_flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)
    if jobs:
        with ThreadPoolExecutor(max_workers=len(jobs)) as ex:
            for cmd, res in zip(jobs, ex.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs)):
                if verbose or res.returncode:
                    sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
                if res.returncode:
                    raise RuntimeError(f"nvcc failed for {cmd[-3]}")
    objs = [os.path.join(OBJ, s.replace(".cu", ".o")) for s in SOURCES]
    if force or jobs or _newer(LIB, objs):
        tmp = LIB + f".tmp{os.getpid()}"
        subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs +
                              ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
