"""Build the CUDA library in-tree: paper_2609_26077_b200/libfmm_b200.so (sm_100a only), and on request its
checked twin libfmm_b200_debug.so (-DFMM_DEBUG: every global store of every kernel is range-checked)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libfmm_b200.so")
SOURCES = ["fmm_api.cu", "fmm_encode.cu", "fmm_gemm.cu", "fmm_stats.cu"]
HEADERS = [os.path.join(CSRC, "fmm_internal.h"), os.path.join(HERE, "..", "include", "fmm.h")]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-cudart", "static"]


OUT_DEBUG = os.path.join(HERE, "libfmm_b200_debug.so")


def _stale(out):
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS + [os.path.join(CSRC, "fmm_ptx.cuh")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    out = OUT_DEBUG if debug else OUT
    if not force and not _stale(out):
        return out
    objs = []
    procs = []
    for s in SOURCES:
        o = os.path.join(CSRC, s.replace(".cu", ".dbg.o" if debug else ".o"))
        cmd = ([NVCC] + FLAGS + (["-DFMM_DEBUG"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) +
               ["-c", os.path.join(CSRC, s), "-o", o])
        procs.append((subprocess.Popen(cmd), cmd))
        objs.append(o)
    for p, cmd in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    subprocess.check_call([NVCC, "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-o", out] + objs)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
