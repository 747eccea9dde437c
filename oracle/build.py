"""Compiles the CPU oracle (plain C, gcc) into oracle/libtoploc_oracle.so.

Test infrastructure: the oracle is the parity reference and the timed CPU
baseline; the CUDA library never links or loads it.
"""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "toploc_oracle.c")
LIBRARY = os.path.join(_HERE, "libtoploc_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIBRARY)
            and os.path.getmtime(LIBRARY) >= os.path.getmtime(SOURCE)):
        return LIBRARY
    tmp = LIBRARY + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", "-pthread",
           SOURCE, "-o", tmp]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    print(build(force=True))
