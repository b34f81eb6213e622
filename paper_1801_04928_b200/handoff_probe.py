"""Builds and runs the stand-alone hand-off probe (``csrc/lf_handoff_probe.cu``).

    python -m paper_1801_04928_b200.handoff_probe

It measures, on the GPU at hand, the pieces a per-layer delta hand-off through L2 is made of: the
latency of one slot load, the time of one poll round of N slots per CTA, and how much gradient-sized
store streams (from the same multiprocessor, from others) add to it.  The single-launch backward
kernels cannot be faster per layer than these figures plus their own arithmetic.
"""
from __future__ import annotations

import os
import subprocess
import sys

from . import build as lfbuild


def main() -> int:
    src = os.path.join(lfbuild.CSRC, "lf_handoff_probe.cu")
    os.makedirs(lfbuild.OBJ, exist_ok=True)
    exe = os.path.join(lfbuild.OBJ, "lf_handoff_probe")
    r = subprocess.run([lfbuild._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17",
                        "-rdc=true", "-o", exe, src], capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        return 1
    return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
