"""Builds libfewbit.so in-tree with nvcc for sm_100a (no other target)."""
from __future__ import annotations

import concurrent.futures
import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(PKG, "libfewbit.so")
OBJ_DIR = os.path.join(PKG, "build")

# (source, object stem, extra flags); the forward kernels are instantiated once per activation
SOURCES = [("fewbit_kernels.cu", "fewbit_kernels", []), ("fewbit_host.cu", "fewbit_host", []),
           ("fewbit_static.cu", "fewbit_static", []), ("fewbit_scan.cu", "fewbit_scan", []), ("fewbit_queue.cu", "fewbit_queue", []),
           ("fewbit_table.cpp", "fewbit_table", [])]
SOURCES += [("fewbit_fwd_inst.cu", f"fewbit_fwd_act{a}", [f"-DFEWBIT_ACT_ID={a}"]) for a in range(9)]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-fvisibility=hidden,-O2", "-I", INCLUDE, "-I", CSRC,
    *os.environ.get("FEWBIT_EXTRA_NVCC_FLAGS", "").split(),
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(INCLUDE, "fewbit.h"))
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs = []
    for src, stem, extra in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ_DIR, stem + ".o")
        if force or _stale(obj, [path] + headers):
            cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", path, "-o", obj]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 4))) as pool:
        for res in pool.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs):
            if verbose and res.stderr:
                print(res.stderr)
            if res.returncode != 0:
                raise RuntimeError("nvcc failed:\n" + " ".join(res.args) + "\n" + res.stdout + res.stderr)
    objs = [os.path.join(OBJ_DIR, stem + ".o") for _, stem, _ in SOURCES]
    if force or jobs or _stale(LIB, objs):
        tmp = LIB + f".{os.getpid()}.tmp"
        subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *objs])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
