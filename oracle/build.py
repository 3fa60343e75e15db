"""Compile the oracle's C source into ``oracle/libbns_oracle.so`` with gcc (test infrastructure)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(HERE, "bns_oracle.c")
LIBRARY = os.path.join(HERE, "libbns_oracle.so")


def build(force: bool = False) -> str:
    """Build the shared library if it is missing or older than its source; return its path.

    ``BNS_ORACLE_LIBRARY`` names a prebuilt library to load instead; only the mutation test sets
    it, to run the pins against a deliberately broken copy of the source."""
    override = os.environ.get("BNS_ORACLE_LIBRARY")
    if override:
        return override
    if not force and os.path.exists(LIBRARY) and os.path.getmtime(LIBRARY) >= os.path.getmtime(SOURCE):
        return LIBRARY
    compile_source(SOURCE, LIBRARY)
    return LIBRARY


def compile_source(source: str, library: str) -> None:
    tmp = library + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", tmp, source, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, library)


if __name__ == "__main__":
    print(build(force=True))
