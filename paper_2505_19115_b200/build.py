"""Compile the CUDA sources into paper_2505_19115_b200/libnvfp4.so (sm_100a only)."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
OUT = os.path.join(HERE, "libnvfp4.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def sources():
    return sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))


def _deps():
    return (sources() + glob.glob(os.path.join(HERE, "csrc", "*.cuh")) + glob.glob(os.path.join(HERE, "csrc", "*.h"))
            + [os.path.join(ROOT, "include", "nvfp4.h")])


def _compile(out: str, srcs, defines=(), verbose: bool = False) -> str:
    cmd = [NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
           "--fmad=false",  # every fp32 operation of the quantizer is a single rounding
           "-I", os.path.join(ROOT, "include"), "-o", out] + [f"-D{d}" for d in defines] + list(srcs)
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return out


def _fresh(out: str) -> bool:
    return os.path.exists(out) and all(os.path.getmtime(out) >= os.path.getmtime(d) for d in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and _fresh(OUT):
        return OUT
    return _compile(OUT, sources(), verbose=verbose)


# Debug build of the same sources with the GEMM's per-role cycle account compiled in (microbench.py gemm_account).
ACCOUNT_OUT = os.path.join(HERE, "libnvfp4_account.so")


def build_account(force: bool = False) -> str:
    if not force and _fresh(ACCOUNT_OUT):
        return ACCOUNT_OUT
    return _compile(ACCOUNT_OUT, sources(), defines=("NVFP4_GEMM_ACCOUNT",))


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
