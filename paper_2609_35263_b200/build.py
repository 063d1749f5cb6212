"""Builds libwpp.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libwpp.so")
SOURCES = ["wpp_plan.cpp", "wpp_waves.cpp", "wpp_hints.cu", "wpp_api.cu", "wpp_append_combine.cu", "wpp_attention.cu", "wpp_attention_small.cu",
           "wpp_kda.cu", "wpp_kda_tc.cu"]
HEADERS = ["wpp_host.h", "wpp_plan_format.h", "wpp_device.h", "wpp_ptx.cuh", os.path.join("..", "..", "include", "wpp.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", shutil.which("nvcc")):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, defines=(), out: str = None) -> str:
    """Compile the library; `defines` (a list of NAME=VALUE strings) and `out` build a variant beside it."""
    if out is None and not force and not is_stale():
        return LIB
    target = out or LIB
    tmp = target + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default", "-cudart", "static",
           "-x", "cu"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [f"-D{d}" for d in defines]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, target)
    return target


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
