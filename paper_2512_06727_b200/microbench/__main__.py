"""Build and run the stand-alone measurements of the tile kernel's building blocks (pair_ops.cu) on the current GPU.

    python -m paper_2512_06727_b200.microbench

Needs nvcc and one B200; prints the program's output.  The binary is written beside the source.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(os.path.dirname(HERE), "csrc")


def main() -> int:
    exe = os.path.join(HERE, "pair_ops")
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-I", CSRC, "-o", exe,
           os.path.join(HERE, "pair_ops.cu"), "-lcuda"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        return r.returncode
    return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
