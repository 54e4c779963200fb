"""Builds the small CUDA helpers that only tests use (never part of libadore.so)."""
import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))


def build_wait_probe(force: bool = False) -> str:
    """Compiles wait_probe.cu for sm_100a into wait_probe.so next to it and returns the path."""
    src, lib = os.path.join(HERE, "wait_probe.cu"), os.path.join(HERE, "wait_probe.so")
    dep = os.path.join(os.path.dirname(os.path.dirname(HERE)), "paper_2407_02328_b200", "csrc", "mbarrier.cuh")
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= max(os.path.getmtime(src), os.path.getmtime(dep)):
        return lib
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    res = subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--shared",
                          "-Xcompiler", "-fPIC", "-cudart", "static", "-o", lib, src], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib
