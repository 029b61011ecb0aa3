"""Stand-alone hardware probes (sm_100a) behind the roofline discussion of the tile bodies.

    python -m paper_2609_22335_b200.probes [l2_to_smem|mma_issue|mbarrier_wait ...]

Each probe is one small CUDA program, built with nvcc into a temporary directory and run on the
current GPU; its output is printed as is.  Nothing of the hot path depends on them.

* ``l2_to_smem``   bulk-copy throughput from an L2-resident region into shared memory, per SM,
                   for several numbers of CTAs per SM, pipeline depths and copy sizes
* ``mma_issue``    cycles one thread needs to issue batches of ``tcgen05.mma`` (M = 128, K = 16,
                   N = 16..256) plus a commit, and cycles until the batch has completed
* ``mbarrier_wait`` cycles of one ``mbarrier.try_wait`` / ``test_wait`` on a phase that completed
                   long before, for one thread and for all 128 threads of a block

Every wait in the probes is bounded.
"""
from __future__ import annotations

import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))
PROBES = ["l2_to_smem", "mma_issue", "mbarrier_wait"]


def run(name: str) -> str:
    """Builds and runs one probe; returns its standard output."""
    if name not in PROBES:
        raise ValueError(f"unknown probe {name!r}; one of {PROBES}")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, name)
        subprocess.run([nvcc, "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-o", exe, os.path.join(HERE, name + ".cu")],
                       check=True)
        return subprocess.run([exe], check=True, capture_output=True, text=True, timeout=300).stdout


def main(argv=None):
    names = (argv if argv is not None else sys.argv[1:]) or PROBES
    for n in names:
        print(f"== {n}")
        print(run(n), end="")


if __name__ == "__main__":
    main()
