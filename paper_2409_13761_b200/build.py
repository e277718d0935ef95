"""Build libkdn.so (CUDA, sm_100a only) in-tree with nvcc.  ``python -m paper_2409_13761_b200.build``."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libkdn.so")
SOURCES = [os.path.join(CSRC, "kdn.cu"), os.path.join(CSRC, "kdn_shell.cu")]
DEPS = SOURCES + [os.path.join(CSRC, "kdn_kernels.cuh"), os.path.join(CSRC, "kdn_td.cuh"), os.path.join(ROOT, "include", "kdn.h")]


def nvcc_path() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libkdn.so cannot be built")


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(d) <= t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "-I", os.path.join(ROOT, "include"),
           "-I", CSRC, "-o", tmp] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


def cuda_home() -> str:
    return os.path.dirname(os.path.dirname(nvcc_path()))


def build_example(name: str, out_dir: str) -> str:
    """Compile examples/<name>.c (plain C99 against include/kdn.h) and link it with libkdn.so; returns the executable."""
    build()
    src = os.path.join(HERE, "examples", name + ".c")
    exe = os.path.join(out_dir, name)
    cc = shutil.which("gcc") or shutil.which("cc")
    if not cc:
        raise RuntimeError("no C compiler found")
    cuda = cuda_home()
    subprocess.run([cc, "-std=c99", "-O2", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                    src, "-o", exe, "-L", HERE, "-lkdn", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                    "-Wl,-rpath," + HERE, "-Wl,-rpath," + os.path.join(cuda, "lib64")], check=True)
    return exe


def example_env() -> dict:
    env = dict(os.environ)
    env["LD_LIBRARY_PATH"] = HERE + os.pathsep + os.path.join(cuda_home(), "lib64") + os.pathsep + env.get("LD_LIBRARY_PATH", "")
    return env


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
