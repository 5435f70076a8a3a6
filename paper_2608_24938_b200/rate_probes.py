"""Builds and runs the tensor-pipe / copy rate probes (csrc/probes/tensor_pipe_probes.cu) on the current GPU.

A development tool: it measures what the grouped GEMMs' design rests on (the rate of tcgen05.mma by shape and CTA
group, what concurrent L2 -> shared-memory traffic does to the clock, the cost of a one-thread TMA producer loop).

    python -m paper_2608_24938_b200.rate_probes [all|mma|pair|copy]
"""
import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def main():
    what = sys.argv[1] if len(sys.argv) > 1 else "all"
    exe = os.path.join(tempfile.mkdtemp(prefix="exfold_probes_"), "tensor_pipe_probes")
    src = os.path.join(HERE, "csrc", "probes", "tensor_pipe_probes.cu")
    subprocess.run([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-o", exe, src, "-lcuda"],
                   check=True)
    sys.exit(subprocess.run([exe, what]).returncode)


if __name__ == "__main__":
    main()
