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
SOURCES = ["sar_gat.cu", "sar_lean_fwd_f32.cu", "sar_lean_fwd_bf16.cu", "sar_lean_bwd_dst_f32.cu", "sar_lean_bwd_dst_bf16.cu", "sar_lean_bwd_src_f32.cu", "sar_lean_bwd_src_bf16.cu",
           "sar_graph.cu", "sar_host.cu", "sar_noalloc.cu", "sar_storing.cu",
           "sar_glue.cu", "sar_norm.cu", "sar_linear.cu", "sar_rgcn.cu"]
NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
    "-DSAR_BUILT_FOR_SM=100", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]
# extra flags for the lean-kernel translation units only (tuning experiments), e.g. SAR_LEAN_NVCC_EXTRA="-DSAR_LEAN_EXPERIMENT"
LEAN_EXTRA = os.environ.get("SAR_LEAN_NVCC_EXTRA", "").split()


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
    raise RuntimeError("sar_linear.cu needs a CUTLASS / CuTe header tree with sm100 support (cute/arch/mma_sm100_umma.hpp): "
                       "none found in this Python environment's flashinfer or tilelang packages; set CUTLASS_PATH to the "
                       "root of a CUTLASS checkout (the directory that holds include/ and tools/util/include/)")


def _deps(path: str, seen=None) -> list:
    """The file and every header of this library it includes, directly or not (quoted includes only)."""
    import re
    seen = seen if seen is not None else []
    if path in seen or not os.path.exists(path):
        return seen
    seen.append(path)
    for inc in re.findall(r'^\s*#\s*include\s+"([^"]+)"', open(path).read(), flags=re.M):
        for base in (os.path.dirname(path), CSRC, os.path.join(ROOT, "include")):
            cand = os.path.join(base, inc)
            if os.path.exists(cand):
                _deps(cand, seen)
                break
    return seen


def _fingerprint(src: str) -> str:
    """Hash of one source file, the headers it reaches and the compiler flags."""
    h = hashlib.sha256()
    for path in sorted(_deps(os.path.join(CSRC, src))):
        h.update(os.path.basename(path).encode())
        h.update(open(path, "rb").read())
    h.update(" ".join(NVCC_FLAGS + (LEAN_EXTRA if src.startswith("sar_lean_") else [])).encode())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the sources whose contents (or headers, or flags) changed since their object was built, in
    parallel, and links libsar.so when any object is new."""
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src):
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        stamp = obj + ".fingerprint"
        fp = _fingerprint(src)
        if not force and os.path.exists(obj) and os.path.exists(stamp) and open(stamp).read() == fp:
            return obj, False
        inc = _cutlass_includes() if src == "sar_linear.cu" else []
        lean = LEAN_EXTRA if src.startswith("sar_lean_") else []
        cmd = [nvcc, *NVCC_FLAGS, *lean, *inc, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        open(stamp, "w").write(fp)
        return obj, True

    with ThreadPoolExecutor(min(len(SOURCES), os.cpu_count() or 4)) as ex:
        results = list(ex.map(compile_one, SOURCES))
    objs = [o for o, _ in results]
    if not force and os.path.exists(LIB) and not any(new for _, new in results):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    r = subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-Xcompiler", "-fPIC"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
