"""Build and run the micro-measurements of csrc/probe_sm100.cu (needs nvcc and a B200):

    python -m paper_2609_39361_b200.probe

Prints the cycles per warp-step of the emulated e4m3 accumulation loop and of its parts, and checks that the
fp64 tensor-core instruction equals a chain of four fma in ascending k.
"""
import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def main() -> int:
    exe = os.path.join(tempfile.mkdtemp(prefix="lamp_probe_"), "probe_sm100")
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "--fmad=false",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(HERE, "csrc"),
           "-o", exe, os.path.join(HERE, "csrc", "probe_sm100.cu")]
    subprocess.run(cmd, check=True)
    return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
