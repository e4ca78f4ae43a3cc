"""Build (nvcc, sm_100a) and run the probes next to this file; prints their tables."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))


def main() -> int:
    rc = 0
    for name, extra in (("int_dispatch", []), ("log_latency", ["-std=c++17", "-I", os.path.join(HERE, "..", "csrc")])):
        src = os.path.join(HERE, name + ".cu")
        exe = os.path.join(HERE, name)
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", *extra, "-o", exe, src])
        rc = rc or subprocess.call([exe])
    return rc


if __name__ == "__main__":
    sys.exit(main())
