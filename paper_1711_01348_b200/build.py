"""Builds libtad.so (host C++ + CUDA for sm_100a) in-tree with nvcc.

The interpreter kernel is compiled once per vector shape (vm_inst.cu with -DTAD_TA / -DTAD_UB),
every shape into an object file of its own, several at a time; the objects land in _build/.
The 16 x 1 shape is compiled twice: once more with 168 registers per thread and blocks of 6 warps.
"""
from __future__ import annotations

import os
import re
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libtad.so")
SOURCES = ["intalg.cpp", "plan.cpp", "codegen.cpp", "contract_gen.cpp", "factor.cpp", "line_gen.cpp", "print.cpp", "api.cpp", "runtime.cu", "contract.cu", "ew.cu", "line.cu"]
HEADERS = ["intalg.h", "plan.h", "gen.h", "program.h", "contract.h", "ew.h", "line.h", "vm.cuh", "vm_shapes.h", "vm_inst.cu",
           os.path.join("..", "..", "include", "tad.h")]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def shapes():
    with open(os.path.join(CSRC, "vm_shapes.h")) as fh:
        return [(int(a), int(b)) for a, b in re.findall(r"M\((\d+), (\d+)\)", fh.read())]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    common = [nvcc, "-std=c++17", "-O3", "-lineinfo", *ARCH, "-Xcompiler", "-fPIC"]
    if verbose:
        common += ["-Xptxas", "-v"]
    jobs = []
    for src in SOURCES:
        jobs.append((common + ["-c", os.path.join(CSRC, src), "-o", os.path.join(OBJ, src + ".o")], src))
    for ta, ub in shapes():
        obj = os.path.join(OBJ, f"vm_{ta}_{ub}.o")
        jobs.append((common + [f"-DTAD_TA={ta}", f"-DTAD_UB={ub}", "-c", os.path.join(CSRC, "vm_inst.cu"), "-o", obj],
                     f"vm_inst {ta}x{ub}"))

    # the 16 x 1 shape once more with 168 registers per thread (kernels whose fused loop runs under per-element masks)
    jobs.append((common + ["-DTAD_TA=16", "-DTAD_UB=1", "-DTAD_RICH_BUILD=1", "-c", os.path.join(CSRC, "vm_inst.cu"),
                           "-o", os.path.join(OBJ, "vm_16_1_rich.o")], "vm_inst 16x1 rich"))

    def run(job):
        cmd, name = job
        res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        return name, res.returncode, res.stdout

    with ThreadPoolExecutor(max_workers=max(1, os.cpu_count() or 1)) as pool:
        results = list(pool.map(run, jobs))
    failed = [r for r in results if r[1] != 0]
    for name, rc, out in results:
        if out and (verbose or rc != 0):
            print(f"--- {name}\n{out}")
    if failed:
        raise RuntimeError("nvcc failed for: " + ", ".join(r[0] for r in failed))
    objs = [job[0][-1] for job in jobs]
    subprocess.check_call([nvcc, *ARCH, "-shared", "-o", LIB, *objs, "-lcudart"])
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
