"""Builds libd2o.so (sm_100a) in-tree with nvcc.  No torch involvement: the library is a plain
C-ABI shared object."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libd2o.so")
LIB_CHECKED = os.path.join(HERE, "libd2o_checked.so")      # the same sources with -DD2O_CHECKED (index checks)
SOURCES = ["d2o_host.cu", "d2o_stats.cu", "d2o_prefill.cu", "d2o_decode.cu", "d2o_full_decode.cu", "d2o_sim_tc.cu", "d2o_colsum_tc.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(out: str, deps) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compiles every .cu file to an object (in _build/) and links libd2o.so next to this file; `checked` builds
    libd2o_checked.so (objects in _build_checked/), whose kernels verify every data-derived index before using it.
    With D2O_SKIP_BUILD=1 in the environment an existing library is used as it is."""
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    if os.environ.get("D2O_SKIP_BUILD") == "1" and os.path.exists(LIB) and not force:
        return LIB
    nvcc = _nvcc()
    bdir = os.path.join(HERE, "_build_checked" if checked else "_build")
    os.makedirs(bdir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "d2o.h"))
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    extra = [f for f in sorted(os.listdir(CSRC)) if f.endswith(".cu") and f not in sources]
    sources += extra
    objs, procs = [], []
    for s in sources:
        src = os.path.join(CSRC, s)
        obj = os.path.join(bdir, s.replace(".cu", ".o"))
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            cmd = [nvcc, *ARCH, "-O3", "-lineinfo", "-std=c++17", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
                   *(["-DD2O_CHECKED"] if checked else []), "-c", src, "-o", obj]
            procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for s, p in procs:
        out, _ = p.communicate()
        with open(os.path.join(bdir, s + ".log"), "w") as f:
            f.write(out)
        if p.returncode != 0:
            failed = True
            sys.stderr.write(out)
        elif verbose:
            sys.stderr.write(out)
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _stale(LIB, objs):
        cmd = [nvcc, *ARCH, "-shared", "-o", LIB, *objs]
        subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
