"""Compile the fp64 CPU oracle (test infrastructure) into ``oracle/liboracle.so`` with gcc."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "convbn_oracle.c")
LIBRARY = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Build the shared library if it is missing or older than its source; return its path.

    Plain ``-O2`` for the generic x86-64 target (the file may be built on one machine and
    loaded on another) and no fast-math, so the arithmetic is IEEE fp64 in loop order.
    """
    if (not force and os.path.exists(LIBRARY)
            and os.path.getmtime(LIBRARY) >= os.path.getmtime(SOURCE)):
        return LIBRARY
    tmp = LIBRARY + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
           "-Wall", "-Wextra", "-o", tmp, SOURCE, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True))
