"""In-tree build of the CUDA library (liblibra.so) for sm_100a with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SO = os.path.join(HERE, "liblibra.so")
SOURCES = ["plan.cu", "attn_fwd.cu", "attn_bwd.cu", "attn_d256.cu", "no_alloc.cu", "vrsp.cu", "tap.cu", "selftest.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _deps():
    out = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    out.append(os.path.join(os.path.dirname(HERE), "include", "libra.h"))
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into liblibra.so next to this file; returns its path."""
    srcs = [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    stale = force or not os.path.exists(SO) or any(os.path.getmtime(d) > os.path.getmtime(SO) for d in _deps())
    if not stale:
        return SO
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("LIBRA_NVCC_EXTRA", "").split()
    objs = []
    procs = []
    for s in srcs:
        o = os.path.join(HERE, "build", os.path.basename(s) + ".o")
        os.makedirs(os.path.dirname(o), exist_ok=True)
        objs.append(o)
        procs.append((s, subprocess.Popen([nvcc, *NVCC_FLAGS, *extra, "-c", s, "-o", o], stdout=subprocess.PIPE,
                                          stderr=subprocess.STDOUT, text=True)))
    for s, p in procs:
        log, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(log)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {s}")
    tmp = SO + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-o", tmp, *objs, "-cudart", "static"])
    os.replace(tmp, SO)
    return SO


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
