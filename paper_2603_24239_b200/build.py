"""Builds libdvm.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every source is compiled to an object of its own, in parallel; the interpreter kernel's template variants are
spread over DVM_INST_GROUPS compilations of csrc/dvm_vm_inst.cu.  Objects live in build/ beside this file and
are rebuilt only when a source or header is newer."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libdvm.so")
SOURCES = ["dvm_host.cpp", "dvm_fuser.cpp", "dvm_launch.cu", "dvm_matmul.cu"]
DVM_INST_GROUPS = 51
HEADERS = ["dvm_format.h", "dvm_internal.h", "dvm_launch.h", "dvm_vm.cuh", "dvm_math.cuh", "dvm_program.h",
           "dvm_vm_variants.h", "dvm_vm_lean.cuh", "dvm_link.h", os.path.join("..", "..", "include", "dvm.h"),
           os.path.join("..", "..", "include", "dvm_fuser.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"] + os.environ.get("DVM_EXTRA_NVCC_FLAGS", "").split()


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _units():
    """(object path, source path, extra flags) of every compilation."""
    units = [(os.path.join(OBJ, os.path.splitext(s)[0] + ".o"), os.path.join(CSRC, s), []) for s in SOURCES]
    for g in range(DVM_INST_GROUPS):
        units.append((os.path.join(OBJ, f"dvm_vm_inst_{g}.o"), os.path.join(CSRC, "dvm_vm_inst.cu"),
                      [f"-DDVM_INST_GROUP={g}"]))
    return units


def _deps_mtime() -> float:
    deps = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.abspath(__file__)]
    return max(os.path.getmtime(d) for d in deps if os.path.exists(d))


def _stale(obj: str, src: str, hdr_time: float) -> bool:
    if not os.path.exists(obj):
        return True
    t = os.path.getmtime(obj)
    return os.path.getmtime(src) > t or hdr_time > t


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    hdr = _deps_mtime()
    return hdr > t or any(os.path.getmtime(src) > t for _, src, _ in _units())


def build(force: bool = False, verbose: bool = False, jobs: int | None = None) -> str:
    """Compiles every CUDA source of the library into paper_2603_24239_b200/libdvm.so."""
    if not force and not needs_build():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    hdr = _deps_mtime()
    todo = [u for u in _units() if force or _stale(u[0], u[1], hdr)]

    def compile_one(unit):
        obj, src, extra = unit
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + extra + ["-c", "-o", obj, src]
        res = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, res

    jobs = jobs or max(1, min(len(todo), os.cpu_count() or 1))
    with ThreadPoolExecutor(max_workers=jobs) as pool:
        for cmd, res in pool.map(compile_one, todo):
            if verbose:
                sys.stderr.write(" ".join(cmd[-4:]) + "\n" + res.stderr)
            if res.returncode != 0:
                raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    link = [_nvcc(), "-shared", "-o", LIB] + [u[0] for u in _units()]
    res = subprocess.run(link, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + " ".join(link) + "\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
