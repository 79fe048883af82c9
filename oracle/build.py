"""Compile the C oracle into ``oracle/libqnn_oracle.so`` (gcc -O2 -fopenmp).

Building the checker is not using it: the build entry point of the repository
calls this so that the GPU machine has the oracle ready for the tests.
"""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "qnn_oracle.c")
LIB = os.path.join(_HERE, "libqnn_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
           "-Wall", "-Wextra", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
