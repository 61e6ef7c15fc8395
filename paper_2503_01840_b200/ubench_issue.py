"""Builds and runs the issue-loop microbenchmark (ubench/issue_loop.cu) on GPU 0.

    python -m paper_2503_01840_b200.ubench_issue

Prints, per tile width N, the cycles one warp spends per instruction of the GEMM main loop (averaged over 64 back-to-back
executions): elect.sync, redux, the tcgen05 fence, a try_wait and a test_wait on a completed mbarrier, tcgen05.commit,
one and four tcgen05.mma (M = 128, K = 16) from an elected lane, four MMAs + commit from an elected lane and from an
`if (lane == 0)` branch, and mbarrier.arrive.expect_tx."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    out = os.path.join(HERE, "_build", "ubench_issue")
    os.makedirs(os.path.dirname(out), exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "--expt-relaxed-constexpr", "-o", out,
                    os.path.join(HERE, "ubench", "issue_loop.cu")], check=True)
    sys.exit(subprocess.run([out]).returncode)


if __name__ == "__main__":
    main()
