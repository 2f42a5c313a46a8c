"""Builds the CUDA library (sm_100a only) in-tree: paper_2609_24197_b200/libhspec.so.

Every kernel file is compiled to its own object (in parallel, and only when it or a header changed) and the objects
are linked into one shared library.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libhspec.so")
SOURCES = ["hspec.cu", "gemm.cu", "gemm_2sm.cu", "attention.cu", "attention_tc.cu", "scan.cu", "elementwise.cu",
           "noalloc.cu", "next_ops.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def build(force=False, verbose=False):
    """Compile every kernel file for sm_100a into one shared library; returns its path."""
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(HERE, "..", "include", "hspec.h"))
    extra = os.environ.get("HSPEC_NVCC_FLAGS", "").split()     # e.g. -DHSPEC_ATTN_TIMING for kernel-internal timing
    if not force and not extra and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest(srcs + headers):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    hdr_time = _newest(headers)
    tag = os.path.join(OBJ, "flags.txt")
    flags_now = " ".join(FLAGS + extra)
    flags_changed = not os.path.exists(tag) or open(tag).read() != flags_now

    def compile_one(src):
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        if (not force and not flags_changed and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(os.path.getmtime(src), hdr_time)):
            return obj, ""
        cmd = [nvcc] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
        return obj, res.stderr

    with ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 4)) as pool:
        results = list(pool.map(compile_one, srcs))
    with open(tag, "w") as f:
        f.write(flags_now)
    if verbose:
        for _, log in results:
            if log:
                print(log)
    res = subprocess.run([nvcc, "--shared", "-o", LIB] + [o for o, _ in results], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
