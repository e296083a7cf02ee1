"""dvm_tensor_extents / dvm_launch_checked: the bytes a program addresses in every tensor, against shape arithmetic
written out here; the checked launch refuses short buffers before it touches the device.  DVM_DEBUG=1 on the GPU."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _numel(shape):
    return int(np.prod(shape))


def test_extents_of_dense_programs():
    c = dvm.encode(dvm.program_from_nodes(wl.program_c1().nodes), [(7, 1531)] * 3)
    assert dvm.tensor_extents(c) == [7 * 1531 * 4] * 4
    c = dvm.encode(dvm.program_from_nodes(wl.program_add_rmsnorm().nodes), [(37, 4096), (37, 4096), (4096,)])
    assert dvm.tensor_extents(c) == [37 * 4096 * 2, 37 * 4096 * 2, 4096 * 2, 37 * 4096 * 2, 37 * 4096 * 2]
    c = dvm.encode(dvm.program_from_nodes(wl.program_masked_softmax().nodes), [(2, 3, 17, 17), (1, 1, 17, 17)])
    assert dvm.tensor_extents(c) == [2 * 3 * 17 * 17 * 2, 17 * 17 * 2, 2 * 3 * 17 * 17 * 2]
    # per-row results, integer outputs, a long row in phases, an empty instance
    p = wl.OpProgram("stats")
    x = p.input("f32", 2)
    p.output(p.reduce("max", x), "f32")
    p.output(p.cast(x, "u8"), "u8")
    c = dvm.encode(dvm.program_from_nodes(p.nodes), [(9, 20000)])
    assert dvm.tensor_extents(c) == [9 * 20000 * 4, 9 * 4, 9 * 20000]
    c = dvm.encode(dvm.program_from_nodes(p.nodes), [(0, 300)])
    assert dvm.tensor_extents(c) == [0, 0, 0]
    c = dvm.encode(dvm.program_from_nodes(wl.program_mlp_gate().nodes), [(300, 512), (512, 256), (512, 256)])
    assert dvm.tensor_extents(c) == [300 * 512 * 2, 512 * 256 * 2, 512 * 256 * 2, 300 * 256 * 2]


def test_extents_of_views_follow_the_strides():
    p = wl.OpProgram("axpy")
    x, y = p.input("bf16", 2), p.input("bf16", 2)
    p.output(p.binary("add", x, y), "bf16")
    hp = dvm.program_from_nodes(p.nodes)
    rows, cols, ld = 300, 100, 304
    # x: the transpose of a [cols, ld] storage; y: rows padded to 128 elements; out: every other row of a larger buffer
    c = dvm.encode(hp, [(rows, cols), (rows, cols)], in_strides=[[1, ld], [128, 1]], out_strides=[[2 * cols, 1]])
    want = [((rows - 1) + (cols - 1) * ld + 1) * 2, ((rows - 1) * 128 + cols) * 2, ((rows - 1) * 2 * cols + cols) * 2]
    assert dvm.tensor_extents(c) == want
    # an expanded operand (stride 0) needs one row only
    c = dvm.encode(hp, [(rows, cols), (rows, cols)], in_strides=[[0, 1], [cols, 1]])
    assert dvm.tensor_extents(c)[0] == cols * 2


def test_checked_launch_refuses_short_buffers_before_the_device():
    c = dvm.encode(dvm.program_from_nodes(wl.program_c1().nodes), [(7, 1531)] * 3)
    full = 7 * 1531 * 4
    with pytest.raises(dvm.DvmError) as ei:
        dvm.launch_checked(c, [0x1000, 0x2000, 0x3000, 0x4000], [full, full, full - 1, full])
    assert ei.value.status == -4      # DVM_ERR_BUFFER_TOO_SMALL; nothing was launched


@pytest.mark.gpu
def test_checked_launch_runs_and_matches_plain_launch():
    prog = wl.program_c1()
    ins = [t.cuda() for t in wl.inputs_c1()]
    c = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins])
    a, b = torch.empty_like(ins[0]), torch.empty_like(ins[0])
    dvm.launch(c, ins + [a])
    dvm.launch_checked(c, ins + [b], [t.numel() * 4 for t in ins + [b]])
    torch.cuda.synchronize()
    assert torch.equal(a, b) and dvm.last_device_status() == 0


@pytest.mark.gpu
def test_debug_mode_checks_on_the_device_and_reports_per_launch():
    """DVM_DEBUG=1 in a fresh process: every launch is preceded by the device-side check of the placed program,
    synchronises, and returns the device status; results equal the normal mode's (parity tests of three kinds of
    launch run under it)."""
    env = dict(os.environ, DVM_DEBUG="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "tests/test_gpu_parity_small.py",
                        "tests/test_gpu_stacked.py", "tests/test_gpu_compare_select.py", "-k", "not config4_launches"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    code = (
        "import torch, dvm_workloads as wl, paper_2603_24239_b200 as dvm\n"
        "ins=[t.cuda() for t in wl.inputs_c1()]\n"
        "c=dvm.encode(dvm.program_from_nodes(wl.program_c1().nodes),[tuple(t.shape) for t in ins])\n"
        "o=torch.empty_like(ins[0]); n0=dvm.launch_count(); dvm.launch(c, ins+[o]); print(dvm.launch_count()-n0)\n")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip().splitlines()[-1] == "2", r.stdout + r.stderr   # check kernel + interpreter
