"""Build and run one of the instruction-rate microbenchmarks that the kernels' design notes quote.

    python -m paper_2512_15176_b200.microbench mma_rate | mma_pair_rate | xu_rate

Each is a standalone CUDA program (nvcc, sm_100a) that prints SM cycles per instruction; needs a B200.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
PKG = os.path.dirname(HERE)
NAMES = ("mma_rate", "mma_pair_rate", "xu_rate")


def main() -> int:
    if len(sys.argv) != 2 or sys.argv[1] not in NAMES:
        print(__doc__)
        return 2
    name = sys.argv[1]
    out_dir = os.path.join(PKG, "_build")
    os.makedirs(out_dir, exist_ok=True)
    exe = os.path.join(out_dir, name)
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-I", os.path.join(PKG, "csrc"),
           "-I", os.path.join(os.path.dirname(PKG), "include"), "-o", exe, os.path.join(HERE, name + ".cu")]
    subprocess.run(cmd, check=True)
    return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
