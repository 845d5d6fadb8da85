"""In-tree build of the CUDA libraries (sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_DIR = os.path.join(HERE, "lib")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]

TARGETS = {
    "libmukv.so": (os.path.join(HERE, "csrc", "mukv.cu"),
                   sorted(glob.glob(os.path.join(HERE, "csrc", "*.cuh")))
                   + [os.path.join(os.path.dirname(HERE), "include", "mukv.h")]),
    "libmukv_synth.so": (os.path.join(HERE, "synth", "synth.cu"), []),
}


def lib_path(name: str) -> str:
    return os.path.join(LIB_DIR, name)


def _stale(out: str, deps) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> None:
    """Compile every CUDA library of the package with nvcc; raises on failure."""
    os.makedirs(LIB_DIR, exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    for name, (src, deps) in TARGETS.items():
        out = lib_path(name)
        if not force and not _stale(out, [src] + deps):
            continue
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", out, src]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose:
            print(r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {name}:\n{r.stdout}\n{r.stderr}")


if __name__ == "__main__":
    import sys
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
