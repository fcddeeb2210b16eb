"""Compile the oracle's C routine with gcc (plain -O2, OpenMP only to spread rows)."""
import os
import subprocess


def build() -> str:
    here = os.path.dirname(os.path.abspath(__file__))
    out = os.path.join(here, "liboracle_attention.so")
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", out,
                           os.path.join(here, "attention_oracle.c"), "-lm"])
    return out


if __name__ == "__main__":
    print(build())
