"""Build the CPU oracle (plain C + OpenMP) into oracle/libconfu_ref.so.

Test infrastructure only: nothing on the product path uses this library.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "confu_ref.c")
HDR = os.path.join(HERE, "confu_ref.h")
LIB = os.path.join(HERE, "libconfu_ref.so")


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its sources."""
    if not force and os.path.exists(LIB):
        newest = max(os.path.getmtime(SRC), os.path.getmtime(HDR))
        if os.path.getmtime(LIB) >= newest:
            return LIB
    cmd = ["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
