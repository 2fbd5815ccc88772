"""Builds libsvlm.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsvlm.so")
BUILD = os.path.join(HERE, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--use_fast_math", "-Xptxas", "-v"]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers():
    inc = os.path.join(os.path.dirname(HERE), "include")
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    hs += [os.path.join(inc, f) for f in os.listdir(inc) if f.endswith(".h")]
    return hs


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(BUILD, exist_ok=True)
    newest_header = max(os.path.getmtime(h) for h in _headers())
    objs, relink = [], force or not os.path.exists(LIB)
    for src in _sources():
        obj = os.path.join(BUILD, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header)
        if stale:
            cmd = ["nvcc", *NVCC_FLAGS, "-c", src, "-o", obj]
            res = subprocess.run(cmd, capture_output=True, text=True)
            with open(obj + ".log", "w") as f:
                f.write(res.stdout + res.stderr)
            if verbose or res.returncode:
                sys.stderr.write(res.stdout + res.stderr)
            if res.returncode:
                raise RuntimeError("nvcc failed on " + src)
            relink = True
    if relink or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        subprocess.check_call(["nvcc", "-shared", "-o", LIB, *objs, "-lcudart"])
    return LIB


def build_trace() -> str:
    """A second library, libsvlm_trace.so, whose decode kernel stamps %globaltimer at the stations of its chain
    (compile-time switch SVLM_DECODE_TRACE in csrc/svlm_decode.cu).  Only the benchmark's decode-trace workload
    loads it; the product library is untouched."""
    build()
    out = os.path.join(HERE, "libsvlm_trace.so")
    src = os.path.join(CSRC, "svlm_decode.cu")
    obj = os.path.join(BUILD, "svlm_decode_trace.o")
    newest = max([os.path.getmtime(src)] + [os.path.getmtime(h) for h in _headers()])
    if not os.path.exists(obj) or os.path.getmtime(obj) < newest:
        res = subprocess.run(["nvcc", *NVCC_FLAGS, "-DSVLM_DECODE_TRACE", "-c", src, "-o", obj], capture_output=True, text=True)
        if res.returncode:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("nvcc failed on the trace build of " + src)
    others = [os.path.join(BUILD, os.path.basename(f)[:-3] + ".o") for f in _sources() if not f.endswith("svlm_decode.cu")]
    if not os.path.exists(out) or any(os.path.getmtime(o) > os.path.getmtime(out) for o in [obj] + others):
        subprocess.check_call(["nvcc", "-shared", "-o", out, obj, *others, "-lcudart"])
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
    if "--trace" in sys.argv:
        print(build_trace())
