"""Compile the CUDA library (sm_100a) into paper_2504_13818_b200/libpods_b200.so with nvcc."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
PKG = os.path.dirname(HERE)
LIB = os.path.join(PKG, "libpods_b200.so")
SOURCES = sorted(glob.glob(os.path.join(HERE, "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(HERE, "*.cuh"))) + [os.path.join(os.path.dirname(PKG), "include", "pods.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "--use_fast_math=false"]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS + [os.path.abspath(__file__)])


CHECKED_LIB = os.path.join(PKG, "libpods_b200_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the library.  ``checked``: the -DPODS_BOUNDS_CHECK variant (every index a kernel computes is compared
    with its extent and reported through the status word), written beside the normal one."""
    if checked:
        return _build(CHECKED_LIB, ["-DPODS_BOUNDS_CHECK"], "_build_checked", verbose)
    if not force and not needs_build():
        return LIB
    return _build(LIB, [], "_build", verbose)


def _build(lib: str, defines, objdir_name: str, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in NVCC_FLAGS if f not in ("--use_fast_math=false", "-shared")] + list(defines)
    if verbose:
        flags += ["-Xptxas", "-v"]
    # one nvcc per source, side by side (the sources share no device symbols), then one link
    objdir = os.path.join(PKG, objdir_name)
    os.makedirs(objdir, exist_ok=True)
    jobs = []
    for src in SOURCES:
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        jobs.append((obj, subprocess.Popen([nvcc] + flags + ["-c", src, "-o", obj])))
    failed = [obj for obj, p in jobs if p.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, "nvcc -c (%s)" % ", ".join(os.path.basename(f) for f in failed))
    tmp = lib + ".tmp%d" % os.getpid()
    subprocess.run([nvcc, "-shared", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a"] + [obj for obj, _ in jobs] + ["-o", tmp], check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
