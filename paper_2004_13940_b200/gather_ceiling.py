"""Runs the gather micro-benchmark (csrc/tools/gather_ceiling.cu): `python -m paper_2004_13940_b200.gather_ceiling`.

It measures how fast the device at hand can gather factor rows of 64 and 512 bytes from tables of
the sizes the workloads have: the ceiling that the stratum SGD and recompute kernels, which are
made of such gathers, can approach.  Needs a CUDA device."""
import subprocess
import sys

from . import build as _build


def main() -> int:
    return subprocess.call([str(_build.build_tools())])


if __name__ == "__main__":
    sys.exit(main())
