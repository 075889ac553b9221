"""Build step: compiles csrc/ampnet.cu and csrc/engine_fast.cu into libampnet.so (in-tree) for sm_100a with nvcc."""
import os
import subprocess

_DIR = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_DIR, "csrc", "ampnet.cu")
SRC_HOST = os.path.join(_DIR, "csrc", "ir_builders.cpp")
SRC_DIRECT = os.path.join(_DIR, "csrc", "engine_fast.cu")
DEPS = [SRC, SRC_HOST, SRC_DIRECT, os.path.join(_DIR, "csrc", "engine.cuh"), os.path.join(_DIR, "csrc", "engine_types.h"),
        os.path.join(os.path.dirname(_DIR), "include", "ampnet.h")]
LIB = os.path.join(_DIR, "libampnet.so")


def up_to_date():
    return os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in DEPS)


def build(force=False, verbose=False):
    if not force and up_to_date():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", tmp, SRC, SRC_DIRECT, SRC_HOST]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
