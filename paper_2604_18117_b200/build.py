"""Builds liblq.so (CUDA kernels + C ABI) for sm_100a with nvcc, in-tree."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liblq.so")
SOURCES = ["lq_api.cu", "lq_quant.cu", "lq_gemm.cu", "lq_gemm_mx.cu", "lq_noalloc.cu", "lq_calibrate.cpp"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-O2,-fopenmp,-ffp-contract=off", "-cudart", "static",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "lq.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


TIMELINE_LIB = os.path.join(HERE, "liblq_timeline.so")


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """Compile every CUDA source into paper_2604_18117_b200/liblq.so; returns its path.
    timeline=True builds liblq_timeline.so instead: the same sources with -DLQ_TIMELINE, whose GEMM kernel
    records per-role clock stamps of CTA 0 (read back with lq_debug_timeline; see timeline.py)."""
    if timeline:
        return _build(TIMELINE_LIB, "_build_timeline", ["-DLQ_TIMELINE"], verbose)
    if not force and not _stale():
        return LIB
    return _build(LIB, "_build", [], verbose)


def _build(lib_path: str, build_subdir: str, extra_flags, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    build_dir = os.path.join(HERE, build_subdir)
    os.makedirs(build_dir, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(build_dir, src + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    # the translation units are independent: compile them side by side
    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    cmd = [nvcc, "-shared", "-cudart", "static", "-Xcompiler", "-fopenmp", "-o", lib_path, *objs, "-lgomp"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, timeline="--timeline" in sys.argv))
