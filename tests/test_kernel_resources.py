"""What the compiler made of the hot kernels (`-Xptxas -v`): the matmul kernel and the lean interpreter must not
spill -- a header change that pushed the matmul epilogue to 255 registers with a stack frame once cost 7 % of the
C5 sweep without failing any other test."""
import os
import re
import shutil
import subprocess

import pytest

CSRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2603_24239_b200", "csrc")
NVCC = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"


def _resources(source, defines=()):
    """kernel name -> (registers, stack bytes, spill stores, spill loads) of every entry function of a source."""
    cmd = [NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xptxas", "-v",
           *defines, "-c", os.path.join(CSRC, source), "-o", os.devnull]
    err = subprocess.run(cmd, capture_output=True, text=True, check=True).stderr
    out, cur = {}, None
    for line in err.splitlines():
        m = re.search(r"Compiling entry function '(\S+)'", line)
        if m:
            cur = m.group(1)
            continue
        m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
        if m and cur:
            out.setdefault(cur, [0, 0, 0, 0])[1:] = [int(m.group(k)) for k in (1, 2, 3)]
        m = re.search(r"Used (\d+) registers", line)
        if m and cur:
            out.setdefault(cur, [0, 0, 0, 0])[0] = int(m.group(1))
    return out


@pytest.mark.skipif(not os.path.exists(NVCC), reason="nvcc not found")
def test_matmul_kernel_keeps_its_registers():
    res = {k: v for k, v in _resources("dvm_matmul.cu").items() if "dvm_mm_kernel" in k}
    assert res, "dvm_mm_kernel not found in the ptxas output"
    for name, (regs, stack, st, ld) in res.items():
        assert stack == 0 and st == 0 and ld == 0, (name, regs, stack, st, ld)
        assert regs <= 200, (name, regs)        # 168 when this was written; 192 threads x 255 would still fit one CTA per SM


@pytest.mark.skipif(not os.path.exists(NVCC), reason="nvcc not found")
def test_lean_interpreter_does_not_spill():
    res = {k: v for k, v in _resources("dvm_vm_inst.cu", ["-DDVM_INST_GROUP=13"]).items() if "lean" in k}
    assert res, "lean kernels not found in the ptxas output"
    for name, (regs, stack, st, ld) in res.items():
        assert stack == 0 and st == 0 and ld == 0, (name, regs, stack, st, ld)
        assert regs <= 128, (name, regs)        # two CTAs of 256 threads per SM
