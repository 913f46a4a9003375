"""Builds libmarlin_b200.so (sm_100a only) next to this file with nvcc.

    python -m paper_2408_11743_b200.build [--force] [--verbose]

The library is built in-tree so that it travels with a snapshot of the repository; nvcc
cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmarlin_b200.so")
SOURCES = ["api.cu", "pack.cu", "pack_sparse.cu", "quantize.cu", "gemm_dense.cu", "gemm_dense_tc.cu", "gemm_tcd.cu"]
HEADERS = [os.path.join(CSRC, "marlin_internal.cuh"), os.path.join(CSRC, "device_utils.cuh"), os.path.join(CSRC, "tc_utils.cuh"), os.path.join(_ROOT, "include", "marlin_b200.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr",
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
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


PTXAS_LOG = os.path.join(_HERE, "ptxas_report.log")


def spill_report():
    """{kernel name: (registers, spill store bytes)} from the last build of the product library, or {} if there is none."""
    import re
    try:
        text = open(PTXAS_LOG).read()
    except OSError:
        return {}
    out = {}
    name = None
    spills = 0
    for line in text.splitlines():
        m = re.search(r"Function properties for (\S+)", line)
        if m:
            name = m.group(1)
            continue
        m = re.search(r"(\d+) bytes spill stores", line)
        if m and name:
            spills = int(m.group(1))
            continue
        m = re.search(r"Used (\d+) registers", line)
        if m and name:
            out[name] = (int(m.group(1)), spills)
            name, spills = None, 0
    return out


def build(force: bool = False, verbose: bool = False, extra_flags=(), out: str = LIB) -> str:
    """Compiles every .cu of the library and links `out`.  `extra_flags` (for example -DMARLIN_TIMING)
    and a different `out` give an instrumented variant beside the product library."""
    if not force and out == LIB and not needs_build():
        return LIB
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o" if out == LIB else ".variant.o"))
        cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, "-I", os.path.join(_ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", obj]
        # the register allocator's report is kept beside the library: spill_report() reads it
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        if verbose:
            print(" ".join(cmd), flush=True)
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    logs = []
    for src, proc in procs:
        log, _ = proc.communicate()
        logs.append(log)
        if proc.returncode != 0 or verbose:
            sys.stderr.write(log)
        failed |= proc.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if out == LIB:
        with open(PTXAS_LOG, "w") as f:
            f.write("".join(logs))
    link = [_nvcc(), "-shared", "-o", out, *objs, "-cudart", "static",
            "-gencode", "arch=compute_100a,code=sm_100a"]
    subprocess.run(link, check=True)
    return out


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
    print(LIB)
