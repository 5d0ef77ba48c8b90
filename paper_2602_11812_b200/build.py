"""Builds the CUDA library in-tree: csrc/*.cu -> paper_2602_11812_b200/libegtp_b200.so (sm_100a only).

nvcc cross-compiles without a GPU.  `python -m paper_2602_11812_b200.build` rebuilds when a
source is newer than the library; `--force` rebuilds always.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
OBJ_DIR = os.path.join(PKG_DIR, "_build")
LIB_PATH = os.path.join(PKG_DIR, "libegtp_b200.so")
SOURCES = ["api.cu", "lmhead_entropy.cu", "pool.cu", "head.cu", "plp.cu", "logits_entropy.cu", "selftest.cu", "head_static.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-cudart", "static",
]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return cand


def _deps():
    out = [os.path.join(ROOT, "include", "egtp.h")]
    for f in os.listdir(CSRC):
        out.append(os.path.join(CSRC, f))
    return out


def sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def up_to_date() -> bool:
    if not os.path.exists(LIB_PATH):
        return False
    t = os.path.getmtime(LIB_PATH)
    return all(os.path.getmtime(p) <= t for p in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB_PATH
    nvcc = _nvcc()
    os.makedirs(OBJ_DIR, exist_ok=True)
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=6) as ex:
        objs = list(ex.map(compile_one, sources()))
    tmp_path = LIB_PATH + f".tmp{os.getpid()}"     # linked aside and renamed: nobody ever sees half a library
    cmd = [nvcc, "-shared", "-cudart", "static", "-o", tmp_path, *objs]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp_path, LIB_PATH)
    return LIB_PATH


def ensure() -> str:
    """build() for callers that only want a usable library: when compiling is impossible here (no nvcc) but a
    library file exists, that file is used as it is; every other failure is raised."""
    try:
        return build()
    except RuntimeError as exc:
        if "nvcc not found" in str(exc) and os.path.exists(LIB_PATH):
            sys.stderr.write(f"warning: {exc}; using the existing {LIB_PATH}\n")
            return LIB_PATH
        raise


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
