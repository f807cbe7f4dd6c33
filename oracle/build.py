"""Compile the CPU oracle (test infrastructure) into a shared library with gcc.

The flags matter for parity: no floating-point contraction (the increment is a
single binary32 multiply, never fused with anything) and no fast-math.
"""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "kahan_oracle.c")
LIBRARY = os.path.join(_HERE, "libkahan_oracle.so")


def build(force: bool = False) -> str:
    """Build liboracle if it is missing or older than its source; return its path."""
    if (not force and os.path.exists(LIBRARY)
            and os.path.getmtime(LIBRARY) >= os.path.getmtime(SOURCE)):
        return LIBRARY
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-Wall", "-Wextra", "-shared", "-fPIC", SOURCE, "-o", LIBRARY + ".tmp", "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(LIBRARY + ".tmp", LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True))
