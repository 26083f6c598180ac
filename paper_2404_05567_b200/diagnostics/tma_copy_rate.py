"""Builds and runs ``tma_copy_rate.cu``: streaming bandwidth of TMA tile copies by copy size and copies in flight.

    python -m paper_2404_05567_b200.diagnostics.tma_copy_rate
"""
import os
import subprocess
import sys

from ..build import CSRC, ROOT, _nvcc

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    out = os.path.join(ROOT, "_build", "tma_copy_rate")
    os.makedirs(os.path.dirname(out), exist_ok=True)
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-I", CSRC,
                           "-I", os.path.join(ROOT, "include"), "-o", out, os.path.join(HERE, "tma_copy_rate.cu"), "-lcuda"])
    sys.exit(subprocess.call([out]))


if __name__ == "__main__":
    main()
