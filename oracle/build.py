"""Compile the CPU oracle (test infrastructure) into oracle/liboracle.so with g++."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ovggt_oracle.cpp")
OUT = os.path.join(HERE, "liboracle.so")


def compile_source(src: str, out: str) -> str:
    """One g++ call: src (which includes ovggt_oracle.h from this folder) -> shared library out."""
    cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-I", HERE,
           "-o", out, src]
    subprocess.run(cmd, check=True)
    return out


def build(force: bool = False) -> str:
    deps = [SRC, os.path.join(HERE, "ovggt_oracle.h")]
    if not force and os.path.exists(OUT) and all(os.path.getmtime(OUT) >= os.path.getmtime(d) for d in deps):
        return OUT
    return compile_source(SRC, OUT)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
