"""Compile the CUDA library in-tree: paper_2507_23387_b200/libsgemm_cube.so (sm_100a only).

nvcc cross-compiles without a GPU.  No fast-math: the split must keep FP16 subnormals and exact
FP32 subtraction / scaling.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsgemm_cube.so")
SOURCES = [os.path.join(CSRC, "sgemm_cube_api.cu")]
DEPS = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + \
       [os.path.join(os.path.dirname(HERE), "include", "sgemm_cube.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    res = subprocess.run([nvcc, *NVCC_FLAGS, *SOURCES, "-o", tmp], capture_output=True, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout)
        print(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
