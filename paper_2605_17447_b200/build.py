"""Build libfastocr.so (hand-written sm_100a CUDA behind a C ABI) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfastocr.so")
SOURCES = ["api.cu", "attn.cu", "topk.cu", "sets.cu", "noalloc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "fastocr.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compile the library. extra_flags / out build a variant (e.g. -DFASTOCR_TRACE) elsewhere."""
    if out is None and not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")] + list(extra_flags)
    lib = out or LIB
    tag = "" if out is None else "." + os.path.basename(out).replace(".so", "")
    if verbose:
        flags += ["-Xptxas", "-v"]
    obj_dir = CSRC if out is None else os.path.dirname(os.path.abspath(out))      # a variant's objects stay beside the variant
    objs = [os.path.join(obj_dir, src.replace(".cu", tag + ".o")) for src in SOURCES]
    procs = [subprocess.Popen([nvcc, *flags, "-c", os.path.join(CSRC, src), "-o", obj]) for src, obj in zip(SOURCES, objs)]
    failed = [src for src, p in zip(SOURCES, procs) if p.wait() != 0]      # the files compile side by side
    if failed:
        raise subprocess.CalledProcessError(1, f"nvcc -c {' '.join(failed)}")
    subprocess.check_call([nvcc, "-shared", "-o", lib, *objs, "-lcudart", "-ldl"])
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
