"""In-tree build of the CUDA library (sm_100a only).

Every ``csrc/*.cu`` is compiled to an object file under ``_build/`` and linked into
``libb2gemm.so`` beside this file.  Objects are rebuilt when their source, any header or the
flags change.  ``python -m paper_1611_08035_b200.build`` runs it from a shell.
"""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG_DIR = Path(__file__).resolve().parent
CSRC = PKG_DIR / "csrc"
INCLUDE = PKG_DIR.parent / "include"
BUILD_DIR = PKG_DIR / "_build"
LIB_PATH = PKG_DIR / "libb2gemm.so"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
    # IEEE arithmetic: no fast-math, denormals kept, fused multiply-add on.
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true", "--fmad=true",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stamp(src: Path) -> str:
    h = hashlib.sha256()
    h.update(" ".join(NVCC_FLAGS).encode())
    h.update(src.read_bytes())
    for hdr in sorted(list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + list(INCLUDE.glob("*.h"))):
        h.update(hdr.read_bytes())
    return h.hexdigest()


def _compile(src: Path, verbose: bool) -> Path:
    obj = BUILD_DIR / (src.stem + ".o")
    stamp_file = BUILD_DIR / (src.stem + ".stamp")
    stamp = _stamp(src)
    if obj.exists() and stamp_file.exists() and stamp_file.read_text() == stamp:
        return obj
    cmd = [_nvcc(), *NVCC_FLAGS, "-I", str(INCLUDE), "-I", str(CSRC), "-c", str(src), "-o", str(obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    (BUILD_DIR / (src.stem + ".ptxas.log")).write_text(res.stderr)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src.name}:\n{res.stderr[-8000:]}")
    if verbose:
        sys.stderr.write(f"[b2gemm build] compiled {src.name}\n")
    stamp_file.write_text(stamp)
    return obj


def build(verbose: bool = False, force: bool = False) -> Path:
    """Compile and link ``libb2gemm.so``; returns its path."""
    BUILD_DIR.mkdir(exist_ok=True)
    if force:
        for f in BUILD_DIR.glob("*.stamp"):
            f.unlink()
    sources = sorted(CSRC.glob("*.cu"))
    if not sources:
        raise RuntimeError("no CUDA sources found")
    # objects, stamps and logs of sources that no longer exist would be linked / reported: drop them
    stems = {src.stem for src in sources}
    stale = False
    for f in list(BUILD_DIR.iterdir()):
        stem = f.name.split(".")[0]
        if f.suffix in (".o", ".stamp", ".log") and stem not in stems:
            f.unlink()
            stale = True
    force = force or stale
    with ThreadPoolExecutor(max_workers=min(8, len(sources))) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose), sources))
    newest = max(o.stat().st_mtime for o in objs)
    if force or not LIB_PATH.exists() or LIB_PATH.stat().st_mtime < newest:
        cmd = [_nvcc(), "-shared", "-o", str(LIB_PATH), *map(str, objs), "-lcudart"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"link failed:\n{res.stderr[-4000:]}")
        if verbose:
            sys.stderr.write(f"[b2gemm build] linked {LIB_PATH.name}\n")
    return LIB_PATH


def ptxas_report() -> str:
    """Concatenated ``-Xptxas -v`` output of the last build (registers, spills, shared memory)."""
    return "\n".join(p.read_text() for p in sorted(BUILD_DIR.glob("*.ptxas.log")))


def ptxas_summary() -> str:
    """Markdown table of every kernel of the last build: registers, static shared memory, stack and spill bytes.

    Parsed from the ``-Xptxas -v`` logs of the build; kernels that differ only in their transposition or
    alignment template flags and use the same resources share a row.  The paper's spilling experiment
    (Section 6.3) makes "no spills" a hard rule for the micro-kernel; the last column shows it holds.
    """
    import re
    rows = {}
    for log in sorted(BUILD_DIR.glob("*.ptxas.log")):
        name = None
        spill = stack = None
        for line in log.read_text().splitlines():
            m = re.search(r"Compiling entry function '([^']+)'", line)
            if m:
                name = m.group(1)
                continue
            m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
            if m and name:
                stack, spill = int(m.group(1)), int(m.group(2)) + int(m.group(3))
                continue
            m = re.search(r"Used (\d+) registers(?:, used \d+ barriers)?(?:, (\d+) bytes smem)?", line)
            if m and name:
                regs, smem = int(m.group(1)), int(m.group(2) or 0)
                pretty = _demangle(name)
                key = (log.stem.replace(".ptxas", ""), _fold_flags(pretty), regs, smem, stack or 0, spill or 0)
                rows[key] = rows.get(key, 0) + 1
                name = None
    out = ["| source file | kernel (template flags folded: `*` = any of true/false) | instances | registers | "
           "static smem B | stack B | spill B |", "|---|---|---|---|---|---|---|"]
    for (src, kern, regs, smem, stack, spill), count in sorted(rows.items()):
        out.append(f"| {src}.cu | `{kern}` | {count} | {regs} | {smem} | {stack} | {spill} |")
    total = sum(rows.values())
    spilled = sum(c for k, c in rows.items() if k[5] or k[4])
    out.append("")
    out.append(f"{total} kernels, {spilled} with a stack frame or spills.")
    return "\n".join(out)


def _demangle(name: str) -> str:
    exe = shutil.which("cu++filt") or shutil.which("c++filt")
    if not exe:
        return name
    res = subprocess.run([exe, name], capture_output=True, text=True)
    text = res.stdout.strip() or name
    import re
    text = re.sub(r"\(anonymous namespace\)::|<unnamed>::", "", text)
    text = re.sub(r"^void ", "", text)
    text = re.sub(r"\((?:int|bool|unsigned int|b2::Layout)\)", "", text)  # casts inside template argument lists
    depth = 0
    for i in range(len(text) - 1, -1, -1):  # drop the parameter list: the last top-level parenthesis group
        if text[i] == ")":
            depth += 1
        elif text[i] == "(":
            depth -= 1
            if depth == 0:
                text = text[:i]
                break
    return text.replace("b2::", "")


def _fold_flags(pretty: str) -> str:
    import re
    return re.sub(r"\b(true|false)\b", "*", pretty)  # cu++filt prints bool template arguments as true/false


if __name__ == "__main__":
    build(verbose=True, force="--force" in sys.argv)
    if "--ptxas" in sys.argv:
        print(ptxas_report())
    if "--ptxas-summary" in sys.argv:
        print(ptxas_summary())
