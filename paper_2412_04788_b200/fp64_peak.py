"""Builds and runs the fp64 latency / throughput micro-benchmark (csrc/fp64_peak.cu) on the current GPU.

    python -m paper_2412_04788_b200.fp64_peak
"""
import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))


def main() -> int:
    src = os.path.join(HERE, "csrc", "fp64_peak.cu")
    exe = os.path.join(tempfile.mkdtemp(prefix="fp64_peak_"), "fp64_peak")
    cmd = [os.environ.get("NVCC", "nvcc"), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-fmad=false",
           "-o", exe, src]
    subprocess.run(cmd, check=True)
    return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
