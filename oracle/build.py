"""Compiles the C oracle into oracle/libkvm_oracle.so (gcc, OpenMP). Test infrastructure only."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "kvm_oracle.c")
LIB = os.path.join(HERE, "libkvm_oracle.so")


def build(force: bool = False) -> str:
    override = os.environ.get("KVM_ORACLE_LIB")  # tests/test_oracle_mutations.py points this at a planted-mistake build
    if override:
        return override
    if (not force) and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
