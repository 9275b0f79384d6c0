"""Compiles csrc/*.cu into libmtrains_b200.so (in-tree) with nvcc for sm_100a."""
import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmtrains_b200.so")


def sources(src_dir: str = CSRC):
    return sorted(glob.glob(os.path.join(src_dir, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > os.path.getmtime(LIB) for d in deps)


def build_library(force: bool = False, verbose: bool = False, out: str = LIB, defines=(), src_dir: str = CSRC) -> str:
    """Compile the library.  `out`, `defines` (e.g. ["MTS_BWD_GROUP1=4"]) and `src_dir` build a
    tuning variant next to the default one."""
    if out == LIB and not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", src_dir,
           "-o", out] + [f"-D{d}" for d in defines] + sources(src_dir)
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return out
