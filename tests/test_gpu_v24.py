"""GPU parity of the 24-elements-per-thread interpreter variant (rows that fill three quarters of a
32-element tile): the five configurations' programs with the setting forced, on aligned, ragged and
misaligned shapes."""
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def v24():
    dvm.set_elems_per_thread(24)
    yield
    dvm.set_elems_per_thread(0)


def _v_of(code):
    import numpy as np
    return int(np.frombuffer(code.bytes(), dtype=np.uint32)[17] >> 24)


@pytest.mark.parametrize("rows,hidden", [(1, 4096), (300, 4096), (257, 1531), (64, 6144), (1000, 72)])
def test_add_rmsnorm(rows, hidden):
    prog = wl.program_add_rmsnorm(hidden)
    ins = wl.inputs_add_rmsnorm(rows, hidden, rows + hidden)
    outs, code = gpu_run(prog, ins)
    assert _v_of(code) == 24
    check(prog, outs, oracle_run(prog, ins))


@pytest.mark.parametrize("B,H,S", [(1, 2, 333), (2, 3, 1400), (1, 4, 768), (1, 1, 17), (1, 2, 6144)])
def test_masked_softmax(B, H, S):
    prog = wl.program_masked_softmax()
    ins = wl.inputs_masked_softmax(B, H, S, S)
    outs, code = gpu_run(prog, ins)
    assert _v_of(code) == 24
    check(prog, outs, oracle_run(prog, ins))


@pytest.mark.parametrize("kind,r,c", [("gelu_affine", 33, 300), ("layernorm", 17, 100), ("sigmoid_mul", 511, 4095),
                                      ("layernorm", 5, 6144), ("gelu_affine", 7, 5000)])
def test_stack_programs_launched_alone(kind, r, c):
    prog = wl.stack_program(kind)
    ins, params = wl.inputs_stack(kind, r, c, r + c)
    p = dvm.program_from_nodes(prog.nodes)
    dev = [t.cuda() for t in ins]
    code = dvm.encode(p, [tuple(t.shape) for t in ins], params)
    assert _v_of(code) == 24
    out = torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")
    dvm.launch(code, dev + [out])
    assert dvm.last_device_status() == 0
    check(prog, [out], oracle_run(prog, ins, params), strict=(kind == "sigmoid_mul"))


def test_c1_and_misaligned_base():
    prog = wl.program_c1()
    ins = wl.inputs_c1()
    outs, code = gpu_run(prog, ins)
    assert _v_of(code) == 24
    check(prog, outs, oracle_run(prog, ins))
    # a base pointer 4 bytes off a 16-byte boundary: the shift comes from the address, full rows wrap around
    hidden, rows = 6144, 9
    p2 = wl.program_add_rmsnorm(hidden)
    ins2 = wl.inputs_add_rmsnorm(rows, hidden, 3)
    pad = [torch.empty(t.numel() + 8, dtype=t.dtype, device="cuda") for t in ins2]
    views = [pd[2:2 + t.numel()].view(t.shape) for pd, t in zip(pad, ins2)]
    for v, t in zip(views, ins2):
        v.copy_(t)
    code2 = dvm.encode(dvm.program_from_nodes(p2.nodes), [tuple(t.shape) for t in ins2])
    outs2 = [torch.full((rows, hidden), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    dvm.launch(code2, views + outs2)
    assert dvm.last_device_status() == 0
    check(p2, outs2, oracle_run(p2, ins2))


def test_stacking_a_24_element_program_is_refused():
    prog = wl.stack_program("sigmoid_mul")
    ins, params = wl.inputs_stack("sigmoid_mul", 8, 100, 1)
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins], params)
    out = torch.empty((8, 100), dtype=torch.float32, device="cuda")
    with pytest.raises(dvm.DvmError) as ei:
        dvm.launch_stacked([code, code], [[t.cuda() for t in ins] + [out]] * 2)
    assert ei.value.status == -3
