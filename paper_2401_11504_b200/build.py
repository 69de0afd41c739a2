"""Build step: compiles csrc/*.cu for sm_100a into libtemplora.so beside this file.

    python -m paper_2401_11504_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  The shared library has no link-time dependency
on the CUDA driver (the one driver call it needs is resolved at run time), so it
loads on a machine without a GPU; kernels of course need a B200.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtemplora.so")
SOURCES = ["api.cu", "tc_gemm.cu", "simt_gemm.cu", "elementwise.cu", "block_ops.cu", "timing.cu", "decode_noalloc.cu", "sm_partition.cu"]


def _nvcc():
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "templora.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force=False, verbose=False):
    """Compile if the library is missing or older than its sources.  Returns its path."""
    if not force and not _stale():
        return LIB
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "--threads", "4", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    cmd += os.environ.get("TEMPLORA_NVCC_FLAGS", "").split()   # e.g. -DTL_SK_CHUNK_MB=16 to try a tuning macro
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
