"""Build the C oracle into ``oracle/libref_gemm.so`` with gcc (``python -m oracle.build``).

Flags: -O2, OpenMP, -ffp-contract=off (one rounding per multiply and per add), no fast-math.
"""
from __future__ import annotations

import shutil
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
SRC = HERE / "ref_gemm.c"
LIB_PATH = HERE / "libref_gemm.so"
CFLAGS = ["-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-Wall"]


def build(force: bool = False) -> Path:
    if not force and LIB_PATH.exists() and LIB_PATH.stat().st_mtime >= max(SRC.stat().st_mtime,
                                                                          Path(__file__).stat().st_mtime):
        return LIB_PATH
    gcc = shutil.which("gcc")
    if gcc is None:
        raise RuntimeError("gcc not found: the oracle cannot be built")
    res = subprocess.run([gcc, *CFLAGS, str(SRC), "-o", str(LIB_PATH), "-lm"], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"gcc failed:\n{res.stderr}")
    if res.stderr.strip():
        sys.stderr.write(res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True))
