"""Compile the CPU oracle (plain C) into oracle/liblpdt_oracle.so.

Test infrastructure only: building the checker is not using it.
Run as `python -m oracle.build` or call build().
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SO = os.path.join(HERE, "liblpdt_oracle.so")
SOURCES = ["lpdt_oracle.c"]
DEPS = SOURCES + ["ren_body.inc"]


def _stale():
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    return any(os.path.getmtime(os.path.join(HERE, s)) > t for s in DEPS)


def build(force=False):
    if not force and not _stale():
        return SO
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wno-unknown-pragmas",
           "-o", SO] + [os.path.join(HERE, s) for s in SOURCES] + ["-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    return SO


if __name__ == "__main__":
    print(build(force=True))
