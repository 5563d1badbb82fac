"""Compile and run the FP32 instruction-mix micro-benchmark (csrc/fp32_mix_bench.cu) on the current GPU.

    python -m paper_1902_06822_b200.fp32_mix

It measures the rates that bound the candidate sweep: scalar and packed (fma.rn.f32x2) forms of the
four-operation evaluation, with and without the saturating min/max, and the cost of folding fp32
partial sums into fp64.
"""
import os
import shutil
import subprocess
import sys
import tempfile

_SRC = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "fp32_mix_bench.cu")


def main() -> int:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    with tempfile.TemporaryDirectory() as d:
        exe = os.path.join(d, "fp32_mix_bench")
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-o", exe, _SRC],
                       check=True)
        return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
