"""Builds libpsattn.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpsattn.so")
SOURCES = ["psattn_api.cu", "psattn_staged.cu", "psattn_noalloc.cu", "psattn_attend_tc.cu", "psattn_measure_mma.cu", "psattn_measure_shared.cu", "psattn_exact_measure.cu", "psattn_project.cu", "psattn_attend64.cu", "psattn_fused.cu", "psattn_probe.cu", "psattn_project_out.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh", ".h"))]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "psattn.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, phase_stamps: bool = False, nvtx: bool = False) -> str:
    """Builds the library.  phase_stamps: a second library, libpsattn_stamps.so, whose kernels record per-phase
    times and their begin and end (-DPSATTN_PHASE_STAMPS); only the benchmark's --phases mode uses it.
    nvtx: a library, libpsattn_nvtx.so, with a named range around every compute entry point (-DPSATTN_NVTX) for
    timeline tools; load it with PSATTN_LIBRARY."""
    if phase_stamps:
        return _build_variant("libpsattn_stamps.so", ["-DPSATTN_PHASE_STAMPS"], ".stamps.o")
    if nvtx:
        return _build_variant("libpsattn_nvtx.so", ["-DPSATTN_NVTX"], ".nvtx.o", ["-ldl"])
    if not force and not needs_build():
        return LIB
    objs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
            print(" ".join(cmd), file=sys.stderr)
        subprocess.check_call(cmd)
        objs.append(obj)
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *objs, "-lcudart"])
    os.replace(tmp, LIB)
    return LIB


def _build_variant(name: str, extra: list, suffix: str, link: list = ()) -> str:
    out = os.path.join(HERE, name)
    objs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", suffix))
        subprocess.check_call([_nvcc(), *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj])
        objs.append(obj)
    tmp = out + ".tmp.%d" % os.getpid()
    subprocess.check_call([_nvcc(), "-shared", "-o", tmp, *objs, "-lcudart", *link])
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, nvtx="--nvtx" in sys.argv))
