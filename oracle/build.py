"""Compile the C oracle into oracle/libpods_oracle.so with gcc (test infrastructure only)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "pods_oracle.c")
LIB = os.path.join(HERE, "libpods_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared",
           "-fno-fast-math", "-ffp-contract=off", "-Wall", "-Wextra",
           SRC, "-o", LIB + ".tmp%d" % os.getpid(), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(LIB + ".tmp%d" % os.getpid(), LIB)   # atomic: safe under concurrent builders
    return LIB


if __name__ == "__main__":
    print(build(force=True))
