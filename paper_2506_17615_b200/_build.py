"""In-tree build of the CUDA library for sm_100a (nvcc cross-compiles without a GPU)."""
import fcntl
import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = [os.path.join(_HERE, "csrc", "equarx_host.cu")]
DEPENDS = SOURCES + [os.path.join(_HERE, "csrc", "equarx_kernels.cuh"),
                     os.path.join(os.path.dirname(_HERE), "include", "equarx.h")]
LIB = os.path.join(_HERE, "libequarx.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def find_nvcc():
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return None


def is_stale():
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > built for p in DEPENDS)


def build(force=False, verbose=False):
    """Compile libequarx.so next to this file; returns its path.  EQUARX_LIBRARY=<path> in the
    environment selects an already built library instead (nothing is compiled then)."""
    prebuilt = os.environ.get("EQUARX_LIBRARY")
    if prebuilt and not force:
        if not os.path.exists(prebuilt):
            raise RuntimeError(f"EQUARX_LIBRARY={prebuilt} does not exist")
        return prebuilt
    if not force and not is_stale():
        return LIB
    nvcc = find_nvcc()
    if nvcc is None:
        raise RuntimeError("libequarx.so is missing or out of date and nvcc was not found; "
                           "the CUDA library cannot be built and there is no fallback")
    # several processes (one per GPU under torchrun) may import at once: one builds, the others wait
    with open(LIB + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if force or is_stale():
                tmp = f"{LIB}.{os.getpid()}.tmp"
                cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
                subprocess.run(cmd, check=True)
                os.replace(tmp, LIB)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB
