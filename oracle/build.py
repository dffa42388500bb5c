"""Compile the CPU oracle into oracle/libswarm_oracle.so.

Test infrastructure only: the product path never loads this library.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "swarm_oracle.cpp")
LIB = os.path.join(HERE, "libswarm_oracle.so")


def build(force: bool = False) -> str:
    # SWARM_ORACLE_LIBRARY names an already built library to load instead of the in-tree one. Only the
    # mutation tests set it: they compile copies of the source with a mistake planted in each and check
    # that the pins reject every copy.
    override = os.environ.get("SWARM_ORACLE_LIBRARY")
    if override:
        return override
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-pthread", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
