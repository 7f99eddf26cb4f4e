"""Build libblink.so (CUDA kernels + C ABI) in-tree for sm_100a with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libblink.so")
OBJ = os.path.join(HERE, "_build")


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def sources():
    out = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC)) if f.endswith((".cu", ".cuh", ".h"))]
    out.append(os.path.join(os.path.dirname(HERE), "include", "blink.h"))
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    srcs = sources()
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest(srcs):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    os.makedirs(OBJ, exist_ok=True)
    units = [f for f in sorted(os.listdir(CSRC)) if f.endswith(".cu")]

    def compile_one(f):
        obj = os.path.join(OBJ, f[:-3] + ".o")
        r = subprocess.run([nvcc] + flags + ["-c", os.path.join(CSRC, f), "-o", obj], capture_output=True, text=True)
        return f, obj, r

    # one translation unit per kernel variant family, compiled side by side
    with ThreadPoolExecutor(max_workers=min(len(units), os.cpu_count() or 1)) as ex:
        results = list(ex.map(compile_one, units))
    log = ""
    for f, obj, r in results:
        log += f"==== {f}\n{r.stdout}{r.stderr}"
        if r.returncode != 0:
            sys.stderr.write(log)
            raise RuntimeError(f"nvcc failed compiling {f}")
    r = subprocess.run([nvcc, "-shared", "-o", LIB] + [obj for _, obj, _ in results], capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("nvcc failed linking libblink.so")
    if verbose:
        print(log)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
