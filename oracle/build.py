"""Compile the CPU oracle (plain C + OpenMP) into shared objects next to this file.

Two builds of the same source: double precision (the one parity is judged against) and
single precision (a plain fp32 build; tests show the two agree far
inside the parity tolerance).  TEST INFRASTRUCTURE: the product never loads these.
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "synera_oracle.c")


def lib_path(f32: bool = False) -> str:
    return os.path.join(HERE, "liboracle_f32.so" if f32 else "liboracle_f64.so")


def build(force: bool = False) -> None:
    for f32 in (False, True):
        out = lib_path(f32)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(SRC):
            continue
        cmd = ["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall",
               "-o", out, SRC, "-lm"]
        if f32:
            cmd.insert(1, "-DORC_F32")
        subprocess.check_call(cmd)


if __name__ == "__main__":
    build(force=True)
    print("built", lib_path(False), lib_path(True))
