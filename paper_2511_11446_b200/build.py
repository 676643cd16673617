"""Builds libdiffpro.so (and the input-generator and measurement-probe libraries) in-tree with nvcc for sm_100a.

    python -m paper_2511_11446_b200.build [--force] [--verbose]

No GPU is needed to build. The shared objects land next to this file.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdiffpro.so")
SYNTH_LIB = os.path.join(HERE, "libdpsynth.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]
SOURCES = ["api.cu", "daq.cu", "simt.cu", "gemm_tc.cu", "gemm_ws.cu", "gemm_as.cu", "gemm_bf16.cu", "gemm_grp.cu", "ln.cu"]
SYNTH_SOURCES = ["synth_cuda.cu"]
PROBE_LIB = os.path.join(HERE, "libdpprobe.so")
PROBE_SOURCES = ["peak.cu"]


def _deps():
    hdrs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hdrs.append(os.path.join(os.path.dirname(HERE), "include", "diffpro.h"))
    hdrs.append(os.path.join(os.path.dirname(HERE), "include", "diffpro_probe.h"))
    return hdrs


def _stale(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def _compile(src, verbose):
    obj = os.path.join(OBJ, os.path.basename(src) + ".o")
    if _stale(obj, [src] + _deps()):
        cmd = [NVCC, *ARCH, *FLAGS, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode:
            raise RuntimeError(f"nvcc failed on {src}")
    return obj


def _link(lib, sources, verbose):
    srcs = [os.path.join(CSRC, s) for s in sources]
    with ThreadPoolExecutor(max_workers=len(srcs)) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose), srcs))
    if _stale(lib, objs):
        subprocess.check_call([NVCC, *ARCH, "-shared", "-o", lib, *objs, "-lcudart_static", "-lpthread",
                               "-ldl", "-lrt"])
    return lib


def build(force: bool = False, verbose: bool = False):
    os.makedirs(OBJ, exist_ok=True)
    if force:
        for f in os.listdir(OBJ):
            os.remove(os.path.join(OBJ, f))
    return (_link(LIB, SOURCES, verbose), _link(SYNTH_LIB, SYNTH_SOURCES, verbose),
            _link(PROBE_LIB, PROBE_SOURCES, verbose))


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
