"""Build the CUDA library in-tree: paper_2206_01299_b200/libaq_b200.so (sm_100a only)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = [os.path.join(CSRC, f) for f in ("aq_api.cu", "aq_kernels.cu", "aq_lowbit.cu", "aq_anygroup.cu", "aq_noalloc.cu")]
HEADERS = [os.path.join(CSRC, "aq_internal.h"), os.path.join(CSRC, "aq_device.cuh"),
           os.path.join(os.path.dirname(HERE), "include", "aq_b200.h")]
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libaq_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    # bit-exact fp32: no fused multiply-add, no flush-to-zero, IEEE division
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-Xcompiler", "-fPIC",
]
LINK_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static"]


def nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the sources side by side (one nvcc per file), then links the library."""
    if not force and not stale():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    objs = [os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o") for src in SOURCES]
    extra = ["-Xptxas", "-v"] if verbose else []
    procs = [subprocess.Popen([nvcc()] + NVCC_FLAGS + extra + ["-c", src, "-o", obj]) for src, obj in zip(SOURCES, objs)]
    failed = [src for src, p in zip(SOURCES, procs) if p.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, "nvcc -c " + " ".join(failed))
    subprocess.check_call([nvcc()] + LINK_FLAGS + ["-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
