"""Compile the CUDA library paper_2309_01507_b200/liblpmm.so for sm_100a (in-tree, with nvcc).

-fmad=false keeps every binary32 multiply and add separately rounded in code that does not use the
explicit round-to-nearest intrinsics; division and square root stay IEEE (no fast-math).
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liblpmm.so")
LIB_DEBUG = os.path.join(HERE, "liblpmm_debug.so")   # the checking build (-DLPMM_DEBUG): guard zones + index checks
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC", "-Xfatbin", "-compress-all"]
# (source, extra flags, object name): the step kernels are compiled as four parts side by side
UNITS = [("lpmm_api.cu", [], "api.o"), ("lpmm_quant.cu", [], "quant.o")] + \
        [("lpmm_step.cu", [f"-DLPMM_STEP_PART={p}"], f"step{p}.o") for p in range(4)]


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths.append(os.path.join(os.path.dirname(HERE), "include", "lpmm.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, "build", "debug" if debug else "release")
    os.makedirs(objdir, exist_ok=True)
    variant = ["-DLPMM_DEBUG"] if debug else []
    procs = []
    for src, extra, obj in UNITS:
        cmd = [nvcc, *NVCC_FLAGS, *variant, *extra, *(["-Xptxas", "-v"] if verbose else []), "-c", "-o", os.path.join(objdir, obj),
               os.path.join(CSRC, src)]
        procs.append((cmd, subprocess.Popen(cmd, cwd=CSRC)))
    for cmd, p in procs:
        if p.wait() != 0:
            raise subprocess.CalledProcessError(p.returncode, cmd)
    subprocess.run([nvcc, "-shared", "-cudart", "static", "-o", lib, *[os.path.join(objdir, o) for _, _, o in UNITS]],
                   check=True, cwd=CSRC)
    return lib


def build_all(force: bool = False) -> None:
    build(force=force)
    build(force=force, debug=True)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build(force="--force" in sys.argv, debug=True))
