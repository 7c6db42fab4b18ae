"""Builds ``libcudallm_gemm.so`` in-tree with nvcc for sm_100a.

Usage: ``python -m paper_2506_09092_b200.build [--force] [--verbose]``
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libcudallm_gemm.so")
HEADERS = sorted(glob.glob(os.path.join(os.path.dirname(PKG), "include", "*.h")))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-shared", "-Xcompiler", "-fPIC",
    "-cudart", "static",
]


TABLE_JSON = os.path.join(PKG, "tuned_b200.json")
TABLE_INC = os.path.join(CSRC, "tuned_table.inc")


def write_table_inc() -> None:
    """The packaged search results as C initialisers (``csrc/tuned_table.inc``, generated): one
    ``PackagedEntry`` per record of ``tuned_b200.json``."""
    import json
    entries = {}
    if os.path.exists(TABLE_JSON):
        with open(TABLE_JSON) as f:
            entries = json.load(f)
    lines = ["// generated from tuned_b200.json by build.py -- do not edit"]
    for key in sorted(entries):
        rec = entries[key]
        shape, dtype = key.split(":")
        M, N, K, batch = (int(x) for x in shape.split("x"))
        lines.append('    {%d, %d, %d, %d, %d, %d, "%s", %d, %d},' % (
            M, N, K, batch, 1 if dtype == "bf16" else 0, 1 if rec.get("tma", True) else 0,
            rec["variant"], int(rec.get("group", 0)), int(rec.get("tail", 0))))
    text = "\n".join(lines) + "\n"
    old = open(TABLE_INC).read() if os.path.exists(TABLE_INC) else None
    if old != text:
        with open(TABLE_INC, "w") as f:
            f.write(text)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + HEADERS + [TABLE_INC]


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(f) <= t for f in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every ``csrc/*.cu`` into one shared library; returns its path."""
    write_table_inc()
    if not force and up_to_date():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed: " + " ".join(cmd))
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
