"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libbeagle.so")
CHECKED_LIB_PATH = os.path.join(LIB_DIR, "libbeagle_checked.so")      # the bounds-checking build (tests only)
SOURCES = ["api.cu", "kernels_decode.cu", "kernels_block.cu", "gemm_tc.cu", "gemm_skinny.cu", "attn_decode_tma.cu", "attn_block_umma.cu", "attn_block_bwd_umma.cu", "verify_sample.cu", "block_loss.cu", "block_grad.cu", "rope.cu", "quant_fp8.cu", "tree.cu", "noalloc.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "--use_fast_math", "-Xptxas", "-v",
]


def _newest_source_mtime() -> float:
    t = os.path.getmtime(os.path.join(os.path.dirname(HERE), "include", "beagle.h"))
    for f in os.listdir(CSRC):
        t = max(t, os.path.getmtime(os.path.join(CSRC, f)))
    return t


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compiles every .cu into lib/libbeagle.so (skipped when the library is newer than the sources).
    checked: the bounds-checking build instead (lib/libbeagle_checked.so: -DBEAGLE_BOUNDS_CHECK, relocatable device code so
    that every kernel reports into one device word); a test-only library, never loaded by default."""
    os.makedirs(LIB_DIR, exist_ok=True)
    lib_path = CHECKED_LIB_PATH if checked else LIB_PATH
    extra = ["-DBEAGLE_BOUNDS_CHECK", "-rdc=true"] if checked else []
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= _newest_source_mtime():
        return lib_path
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(LIB_DIR, src.replace(".cu", ".checked.o" if checked else ".o"))
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    log = []
    for src, p in procs:
        out, _ = p.communicate()
        log.append(f"== {src}\n{out}")
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{out}")
    link = [nvcc, "-shared", "-o", lib_path, *objs, "-gencode", "arch=compute_100a,code=sm_100a", *(["-rdc=true"] if checked else [])]
    r = subprocess.run(link, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}")
    with open(os.path.join(LIB_DIR, "build_checked.log" if checked else "build.log"), "w") as f:
        f.write("\n".join(log))
    if verbose:
        print("\n".join(log))
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
