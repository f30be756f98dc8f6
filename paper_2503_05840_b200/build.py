"""In-tree build of libslim.so (nvcc, sm_100a only)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libslim.so")
SOURCES = ["slim_api.cu", "slim_generic.cu", "slim_tail.cu", "slim_wkv.cu", "slim_tc.cu", "slim_proj.cu", "slim_xscores.cu", "slim_prompt.cu", "slim_split.cu"]
HEADERS = ["slim_internal.h", "slim_sched.cuh", "slim_ptx.cuh", "slim_combine.cuh"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    deps.append(os.path.join(HERE, "..", "include", "slim.h"))
    return any(os.path.getmtime(p) > t for p in deps)


TRACE_LIB = os.path.join(HERE, "libslim_trace.so")


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """trace=True builds libslim_trace.so, the library with the per-tile instrumentation of the
    tensor-core decode kernel compiled in (-DSLIM_TC_TRACE)."""
    if trace:
        return _build(TRACE_LIB, os.path.join(HERE, "_build", "trace"), ["-DSLIM_TC_TRACE"], verbose)
    if not force and not needs_build():
        return LIB
    return _build(LIB, os.path.join(HERE, "_build"), [], verbose)


def _build(lib_path: str, bdir: str, extra: list, verbose: bool) -> str:
    nvcc = _nvcc()
    os.makedirs(bdir, exist_ok=True)
    objs = []
    procs = []
    for s in SOURCES:
        o = os.path.join(bdir, s.replace(".cu", ".o"))
        cmd = [nvcc] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + \
              ["-c", os.path.join(CSRC, s), "-o", o]
        procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(o)
    for s, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(out)
        if p.returncode:
            raise RuntimeError(f"nvcc failed on {s}")
    cmd = [nvcc, "-shared", "-o", lib_path] + objs + ["-lcudart"]
    r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode:
        sys.stderr.write(r.stdout)
        raise RuntimeError("link failed")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
