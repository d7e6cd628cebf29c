"""Build the CUDA library in-tree: paper_2410_00531_b200/libtpi.so (sm_100a only).

With TPI_TIMELINE=1 in the environment (or ``build(timeline=True)``) a second library, libtpi_timeline.so, is built
with -DTPI_TIMELINE: the decode kernels then stamp a device-side timeline (``bench.py --timeline`` reads it).  The
binding loads that library instead when TPI_TIMELINE=1 is set; the plain library is never instrumented."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libtpi.so")
OUT_TIMELINE = os.path.join(HERE, "libtpi_timeline.so")
SOURCES = ["api.cu", "window.cu", "step_decode.cu", "step_prefill.cu", "inspect.cu", "ops.cu", "static_scratch.cu", "kernels_decode.cu", "kernels_prefill.cu", "gemm_tcgen05.cu", "gemm_tcgen05_pair.cu", "attn_prefill_mma.cu", "attn_prefill_tc.cu", "tp_kernels.cu", "step_tp.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC,-fopenmp,-O3", "--use_fast_math=false"]


def timeline_requested() -> bool:
    return os.environ.get("TPI_TIMELINE", "0") not in ("", "0")


def _stale(out: str) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", f) for f in ("tpi.h", "tpi_ops.h", "tpi_tp.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, timeline: bool | None = None) -> str:
    timeline = timeline_requested() if timeline is None else timeline
    out = OUT_TIMELINE if timeline else OUT
    if not force and not _stale(out):
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")] + (["-DTPI_TIMELINE"] if timeline else [])
    objs = []
    procs = []
    objdir = os.path.join(HERE, "build", "timeline") if timeline else os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *flags, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd)))
        objs.append(obj)
    for src, p in procs:
        if p.wait():
            raise RuntimeError(f"nvcc failed on {src}")
    subprocess.check_call([nvcc, *NVCC_FLAGS[:2], "-shared", "-o", out, *objs, "-Xcompiler", "-fopenmp", "-lgomp"])
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
