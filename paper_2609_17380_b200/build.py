"""Builds libdet.so (CUDA, sm_100a only) in-tree with nvcc.

Flags that matter for the arithmetic: -fmad=false (never contract a*b+c), -ftz=true (flush subnormal
inputs and results), -prec-div=true / -prec-sqrt=true (IEEE division and square root).
"""
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_DIR, "csrc")
OUT = os.path.join(_DIR, "libdet.so")
SOURCES = ["reduce.cu", "norm_loss.cu", "glue_optim.cu", "igemm.cu", "lsq.cu", "ogemm.cu", "attn.cu", "attn_pv8.cu", "headops.cu", "sum_static.cu", "lmhead_v2.cu", "attn_v2.cu"]
HEADERS = ["common.cuh", "internal.h", "ogemm_core.cuh", "tc05.cuh", "v2_slice.cuh", os.path.join("..", "..", "include", "det.h"),
           os.path.join("..", "..", "include", "det_test.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
              "-ftz=true", "-prec-div=true", "-prec-sqrt=true", "-Xcompiler", "-fPIC"]


def _nvcc():
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False):
    hdrs = [os.path.join(CSRC, h) for h in HEADERS]
    objdir = os.path.join(_DIR, "build")
    os.makedirs(objdir, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(src):
        s = os.path.join(CSRC, src)
        o = os.path.join(objdir, src.replace(".cu", ".o"))
        if force or _stale(o, [s] + hdrs):
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if r.returncode != 0:
                raise RuntimeError("nvcc failed for %s:\n%s" % (src, r.stderr))
            if verbose:
                print(r.stderr)
        return o

    with ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    if force or _stale(OUT, objs):
        cmd = [nvcc, "-shared", "-o", OUT] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-lcudart_static", "-ldl",
                                                     "-lrt", "-lpthread"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n%s" % r.stderr)
    return OUT


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
