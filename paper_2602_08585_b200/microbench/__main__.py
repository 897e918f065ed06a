"""Builds and runs the epilogue micro-benchmark: `python -m paper_2602_08585_b200.microbench` (one B200)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
PKG = os.path.dirname(HERE)
ROOT = os.path.dirname(PKG)
EXE = os.path.join(HERE, "epilogue_rates")


def build() -> str:
    src = os.path.join(HERE, "epilogue_rates.cu")
    deps = [src] + [os.path.join(PKG, "csrc", f) for f in ("score_chunks.cuh", "tc_ptx.cuh", "common.cuh")]
    if not os.path.exists(EXE) or any(os.path.getmtime(d) > os.path.getmtime(EXE) for d in deps):
        subprocess.run([os.environ.get("NVCC", "nvcc"), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
                        "-std=c++17", "-use_fast_math", "-I", os.path.join(ROOT, "include"), "-I",
                        os.path.join(PKG, "csrc"), "-o", EXE, src], check=True)
    return EXE


if __name__ == "__main__":
    exe = build()
    if "--build-only" not in sys.argv:
        sys.exit(subprocess.run([exe]).returncode)
