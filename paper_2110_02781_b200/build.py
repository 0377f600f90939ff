"""Compile the CUDA library in-tree: `python -m paper_2110_02781_b200.build`.

Produces paper_2110_02781_b200/libftpipe.so for sm_100a.  nvcc cross-compiles, so no GPU is
needed to build.  Objects are rebuilt only when a source or header is newer.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libftpipe.so")
OBJ = os.path.join(HERE, "_build")
SOURCES = ["partition.cpp", "model.cu", "gemm_f32.cu", "elem.cu", "gemm_tc.cu", "gemm_tc32.cu", "stem.cu", "noalloc.cu"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC,-Wall,-ffp-contract=off", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def build(verbose=False, force=False, timeline=False):
    """timeline=True: the measurement variant (-DFTP_TIMELINE, see csrc/launch.cuh) as libftpipe_timeline.so; load it by
    setting FTPIPE_LIB to its path."""
    global OBJ, OUT
    if timeline:
        OBJ, OUT = os.path.join(HERE, "_build_timeline"), os.path.join(HERE, "libftpipe_timeline.so")
        FLAGS.append("-DFTP_TIMELINE")
    os.makedirs(OBJ, exist_ok=True)
    srcs = SOURCES
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(ROOT, "include", "ftpipe.h"))
    hdr_time = _newest(headers)
    jobs = []
    objs = []
    for s in srcs:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ, s + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_time):
            cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", src, "-o", obj]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    with ThreadPoolExecutor(max_workers=4) as ex:
        for cmd, r in ex.map(run, jobs):
            if verbose or r.returncode:
                sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
            if r.returncode:
                raise RuntimeError("nvcc failed on " + cmd[-3])
    if jobs or not os.path.exists(OUT):
        cmd = [NVCC, "-shared", "-o", OUT] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return OUT


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, force="-f" in sys.argv, timeline="--timeline" in sys.argv))
