"""Builds libdirotq.so in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdirotq.so")
SOURCES = ["api.cu", "prepare.cu", "rotate_quant.cu", "w4a4_gemm.cu", "peak.cu", "noalloc.cu", "nvfp4_gemm.cu", "w4a8_gemm.cu", "gptq.cu", "calib.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


# The fallback build: the W4A4 group sums on the integer tensor-core path (see kI8Path in csrc/common.h).  Same sources,
# same interface; the binding loads it instead of libdirotq.so when DIROTQ_LIBRARY names it.
LIB_I8 = os.path.join(HERE, "libdirotq_i8.so")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "dirotq.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def _build(lib: str, build_dir: str, defines: list[str], force: bool, verbose: bool) -> str:
    if not force and not needs_build(lib):
        return lib
    objs = []
    procs = []
    os.makedirs(build_dir, exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(build_dir, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, *defines, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = lib + f".{os.getpid()}.tmp"
    subprocess.check_call([_nvcc(), "-Wno-deprecated-gpu-targets", "-shared", "-o", tmp, *objs, "-cudart", "static", "-Xlinker", "--no-undefined",
                           "-lpthread", "-ldl", "-lrt"])
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    return _build(LIB, os.path.join(HERE, "_build"), [], force, verbose)


def build_i8(force: bool = False, verbose: bool = False) -> str:
    return _build(LIB_I8, os.path.join(HERE, "_build_i8"), ["-DDIROTQ_I8_PATH"], force, verbose)


# The diagnostic build: block 0 of every kernel stamps the SM clock at marked points of its roles into spare slots of the workspace's
# status block (TRACE_CLK in csrc/ptx.cuh; the slot map is at each kernel's first stamp).  paper_2605_16732_b200/trace.py reads it.
LIB_TRACE = os.path.join(HERE, "libdirotq_trace.so")


def build_trace(force: bool = False, verbose: bool = False) -> str:
    return _build(LIB_TRACE, os.path.join(HERE, "_build_trace"), ["-DDIROTQ_TRACE"], force, verbose)


if __name__ == "__main__":
    fn = build_i8 if "--i8" in sys.argv else build_trace if "--trace" in sys.argv else build
    print(fn(force="--force" in sys.argv, verbose="-v" in sys.argv))
