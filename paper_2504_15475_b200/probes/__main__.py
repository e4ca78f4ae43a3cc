"""Build (nvcc, sm_100a) and run the probes next to this file; prints their tables."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))


def main() -> int:
    src = os.path.join(HERE, "int_dispatch.cu")
    exe = os.path.join(HERE, "int_dispatch")
    subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-o", exe, src])
    return subprocess.call([exe])


if __name__ == "__main__":
    sys.exit(main())
