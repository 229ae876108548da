"""Builds the test-only CUDA probes of this folder (nvcc, sm_100a) into shared objects next to
their sources.  They are test infrastructure: nothing in the package loads them."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(os.path.dirname(_HERE))


def build(name: str = "wait_probe", force: bool = False) -> str:
    src = os.path.join(_HERE, name + ".cu")
    lib = os.path.join(_HERE, "lib" + name + ".so")
    deps = [src, os.path.join(_ROOT, "paper_2512_05409_b200", "csrc", "sq_device.cuh")]
    if force or not os.path.exists(lib) or any(os.path.getmtime(d) > os.path.getmtime(lib) for d in deps):
        nvcc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.check_call([nvcc if os.path.exists(nvcc) else "nvcc", "-gencode", "arch=compute_100a,code=sm_100a",
                               "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-shared", "-o", tmp, src])
        os.replace(tmp, lib)
    return lib
