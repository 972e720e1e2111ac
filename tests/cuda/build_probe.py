"""Builds tests/_build/libddd_probe.so from tests/cuda/timeout_probe.cu (nvcc, sm_100a)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
OUT = os.path.join(os.path.dirname(HERE), "_build", "libddd_probe.so")


def build(force: bool = False) -> str:
    src = os.path.join(HERE, "timeout_probe.cu")
    dep = os.path.join(ROOT, "paper_2409_00142_b200", "csrc", "tc_ptx.cuh")
    if not force and os.path.exists(OUT) and os.path.getmtime(OUT) >= max(os.path.getmtime(src), os.path.getmtime(dep)):
        return OUT
    os.makedirs(os.path.dirname(OUT), exist_ok=True)
    tmp = OUT + f".{os.getpid()}.tmp"
    subprocess.run([os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc"), "-gencode", "arch=compute_100a,code=sm_100a",
                    "-lineinfo", "-O3", "-std=c++17", "--shared", "-Xcompiler", "-fPIC", "-cudart", "static",
                    "-I", os.path.join(ROOT, "include"), "-I", os.path.join(ROOT, "paper_2409_00142_b200", "csrc"),
                    "-o", tmp, src], check=True)
    os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    print(build(force=True))
