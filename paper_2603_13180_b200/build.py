"""Builds libmxnorm.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmxnorm.so")
SOURCES = ["mxn_api.cu", "mxn_fwd.cu", "mxn_fwd_fp4.cu", "mxn_bwd.cu", "mxn_transposed.cu"]
HEADERS = ["mxn_device.cuh", "mxn_internal.h", "mxn_row.cuh", "mxn_fwd_common.cuh", "mxn_col.cuh", os.path.join("..", "..", "include", "mxnorm.h")]

# No fast-math and no flush-to-zero: scale selection relies on IEEE division, subnormals and exact
# power-of-two products.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "--ftz=false", "--prec-div=true", "--prec-sqrt=true",
              # no --split-compile: it shortens the build of the forward kernels' file by a third, but changed the code
              # generated for the backward kernel (two registers more, 64.4 -> 68.8 us at [16384, 4096])
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compiles every translation unit in parallel (nvcc -c) and links libmxnorm.so next to this file."""
    if force or _stale():
        import concurrent.futures
        import tempfile
        compile_flags = [f for f in NVCC_FLAGS if f not in ("-shared",)]
        with tempfile.TemporaryDirectory(prefix="mxnorm_build_") as tmpdir:
            def compile_one(src):
                obj = os.path.join(tmpdir, src.replace(".cu", ".o"))
                cmd = ["nvcc", "-c", *compile_flags, *(["-Xptxas", "-v"] if verbose else []), "-o", obj, os.path.join(CSRC, src)]
                res = subprocess.run(cmd, capture_output=True, text=True)
                return src, obj, res
            with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
                results = list(pool.map(compile_one, SOURCES))
            for src, obj, res in results:
                if verbose:
                    sys.stderr.write(res.stderr)
                if res.returncode != 0:
                    raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
            tmp = LIB + f".tmp{os.getpid()}"
            link = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "shared", "-o", tmp,
                    *[obj for _, obj, _ in results]]
            res = subprocess.run(link, capture_output=True, text=True)
            if res.returncode != 0:
                raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
            os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
