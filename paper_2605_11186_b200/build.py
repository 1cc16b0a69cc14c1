"""Compile the CUDA library ``libcats.so`` (sm_100a) in-tree with nvcc."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcats.so")
SOURCES = ["cats_api.cu", "cats_small_kernels.cu", "cats_gemm.cu", "cats_attn.cu"]
HEADERS = ["cats_common.cuh", "cats_kernels.cuh", os.path.join("..", "..", "include", "cats.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--shared", "-cudart", "static"]


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


TIMELINE_LIB = os.path.join(HERE, "libcats_timeline.so")


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """timeline: build the measurement variant (``-DCATS_TIMELINE``, see cats_debug_timeline) as libcats_timeline.so."""
    out = TIMELINE_LIB if timeline else LIB
    if not force and not _stale(out):
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (["-DCATS_TIMELINE"] if timeline else []) + \
        [os.path.join(CSRC, f) for f in SOURCES] + ["-ldl", "-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
