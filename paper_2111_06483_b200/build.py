"""Builds libsar.so (the C-ABI library of include/sar.h) in-tree with nvcc for sm_100a.

    python -m paper_2111_06483_b200.build [--force] [--verbose]

nvcc cross-compiles, so this works on a machine without a GPU.  Sources are compiled in
parallel into csrc/build/*.o and linked into paper_2111_06483_b200/libsar.so.
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(CSRC, "build")
LIB = os.path.join(PKG, "libsar.so")
SOURCES = ["sar_gat.cu", "sar_graph.cu", "sar_host.cu", "sar_noalloc.cu", "sar_glue.cu", "sar_norm.cu", "sar_linear.cu", "sar_rgcn.cu"]
NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
    "-DSAR_BUILT_FOR_SM=100", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _cutlass_includes() -> list:
    """Include paths of a CUTLASS / CuTe header tree with sm100 support (sar_linear.cu instantiates its
    collective templates).  The image vendors one inside the flashinfer package."""
    import site
    roots = list(site.getsitepackages()) + [os.environ.get("CUTLASS_PATH", "")]
    for root in roots:
        for sub in ("flashinfer/data/cutlass", "tilelang/3rdparty/cutlass", ""):
            base = os.path.join(root, sub) if root else ""
            if base and os.path.exists(os.path.join(base, "include", "cute", "arch", "mma_sm100_umma.hpp")):
                return ["-I", os.path.join(base, "include"), "-I", os.path.join(base, "tools", "util", "include")]
    raise RuntimeError("no CUTLASS header tree with sm100 support found (set CUTLASS_PATH)")


def _fingerprint() -> str:
    h = hashlib.sha256()
    for name in sorted(os.listdir(CSRC)):
        path = os.path.join(CSRC, name)
        if os.path.isfile(path):
            h.update(name.encode())
            h.update(open(path, "rb").read())
    h.update(open(os.path.join(ROOT, "include", "sar.h"), "rb").read())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    stamp = os.path.join(OBJ, "fingerprint.txt")
    fp = _fingerprint()
    if not force and os.path.exists(LIB) and os.path.exists(stamp) and open(stamp).read() == fp:
        return LIB
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src):
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        inc = _cutlass_includes() if src == "sar_linear.cu" else []
        cmd = [nvcc, *NVCC_FLAGS, *inc, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with ThreadPoolExecutor(len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    tmp = LIB + f".tmp{os.getpid()}"
    r = subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-Xcompiler", "-fPIC"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, LIB)
    open(stamp, "w").write(fp)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
