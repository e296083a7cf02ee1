"""Reduced rows longer than a tile (Table 1, Sum / Max / Min over a long axis): the program runs in phases over
the column blocks of a row.  Every case against the oracle; maxima and minima bit for bit."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run


def _softmax(dtype):
    p = wl.OpProgram("softmax")
    x = p.input(dtype, 2)
    e = p.unary("exp", p.binary("sub", x, p.reduce("max", x)))
    s = p.reduce("sum", e)
    p.output(p.binary("div", e, s), dtype)
    p.output(s, "f32")
    return p


@pytest.fixture(autouse=True, params=["lean", "general"])
def interpreter(request):
    """Phased programs of the basic instruction set run on the lean interpreter's phased variant; with the lean
    kernel switched off, on the general interpreter: both against the oracle."""
    dvm.set_lean_kernel(request.param == "lean")
    yield request.param
    dvm.set_lean_kernel(True)


def _phases(code):
    for line in dvm.disassemble(code).splitlines():
        if " phases " in line:
            return int(line.split()[-1])
    return 1


def test_long_row_programs_encode_in_phases():
    """Host side only: a softmax needs three passes over a long row (maximum, sum, quotient), an RMSNorm two, a
    plain row sum one; stores sit in the last phase, the scalars are tagged with the phase that completes them."""
    c = dvm.encode(dvm.program_from_nodes(_softmax("bf16").nodes), [(4, 40001)])
    assert dvm.verify(c) == 0 and _phases(c) == 3
    info = dvm.code_info(c)
    assert info["threads_per_row"] == 256 and info["n_tiles"] % (4 * 3) == 0
    text = dvm.disassemble(c)
    assert "@p0 rowmax" in text and "@p1 rowsum" in text and "@p1 store.row" in text and "@p2 store " in text
    c = dvm.encode(dvm.program_from_nodes(wl.program_add_rmsnorm(hidden=50000).nodes), [(3, 50000), (3, 50000), (50000,)])
    assert dvm.verify(c) == 0 and _phases(c) == 2
    p = wl.OpProgram("rowsum")
    p.output(p.reduce("sum", p.input("f32", 2)), "f32")
    c = dvm.encode(dvm.program_from_nodes(p.nodes), [(9, 8193)])
    assert dvm.verify(c) == 0 and _phases(c) == 1 and "@p0 store.row" in dvm.disassemble(c)
    # at 8192 columns a row still fits one tile: no phases
    c = dvm.encode(dvm.program_from_nodes(p.nodes), [(9, 8192)])
    assert "phases" not in dvm.disassemble(c)
    # a phased program is launched on its own: a stacked launch refuses it before it touches the device
    c = dvm.encode(dvm.program_from_nodes(p.nodes), [(9, 8193)])
    with pytest.raises(dvm.DvmError) as ei:
        dvm.launch_stacked([c], [[0x1000, 0x2000]])
    assert ei.value.status == -3


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,rows,cols", [("bf16", 4, 40001), ("f32", 3, 32000), ("bf16", 2, 151936), ("f32", 700, 9001),
                                             ("f32", 1, 8193)])
def test_softmax_over_long_rows(dtype, rows, cols):
    prog = _softmax(dtype)
    x = wl.randn((rows, cols), torch.bfloat16 if dtype == "bf16" else torch.float32, cols, std=3.0)
    outs, code = gpu_run(prog, [x])
    assert _phases(code) == 3
    check(prog, outs, oracle_run(prog, [x]))


@pytest.mark.gpu
def test_layernorm_and_rmsnorm_over_long_rows():
    prog = wl.program_layernorm()
    x = wl.randn((5, 20000), torch.float32, 7, mean=0.5)
    outs, code = gpu_run(prog, [x], [1.0 / 20000])
    assert _phases(code) == 3
    check(prog, outs, oracle_run(prog, [x], [1.0 / 20000]))
    prog = wl.program_add_rmsnorm(hidden=50000)
    ins = wl.inputs_add_rmsnorm(300, 50000, 8)
    outs, code = gpu_run(prog, ins)
    assert _phases(code) == 2
    check(prog, outs, oracle_run(prog, ins))


@pytest.mark.gpu
def test_row_statistics_of_long_rows_are_exact_where_they_can_be():
    p = wl.OpProgram("stats")
    x = p.input("f32", 2)
    p.output(p.reduce("max", x), "f32")
    p.output(p.reduce("min", x), "f32")
    p.output(p.reduce("sum", p.unary("abs", x)), "f32")
    x_t = wl.randn((37, 100003), torch.float32, 9)
    outs, code = gpu_run(p, [x_t])
    want = oracle_run(p, [x_t])
    assert np.array_equal(wl.to_f64(outs[0]), want[0]) and np.array_equal(wl.to_f64(outs[1]), want[1])
    # 100003 non-negative addends in fp32, pairwise inside a tile and tile by tile across the row
    assert np.max(np.abs(wl.to_f64(outs[2]) - want[2]) / want[2]) <= 2e-6


@pytest.mark.gpu
def test_logits_with_bias_and_temperature_then_log_softmax():
    """A vocabulary-sized row with a row-vector operand (loaded per column block) and a per-row scalar input:
    log-softmax((x + b) * t)."""
    p = wl.OpProgram("log_softmax")
    x, b, t = p.input("bf16", 2), p.input("f32", 2), p.input("f32", 2)
    z = p.binary("mul", p.binary("add", x, b), t)
    d = p.binary("sub", z, p.reduce("max", z))
    lse = p.unary("log", p.reduce("sum", p.unary("exp", d)))
    p.output(p.binary("sub", d, lse), "f32")
    p.output(lse, "f32")
    ins = [wl.randn((6, 128257), torch.bfloat16, 1, std=2.0), wl.randn((1, 128257), torch.float32, 2),
           wl.uniform((6, 1), torch.float32, 3, lo=0.5, hi=1.5)]
    outs, code = gpu_run(p, ins)
    assert _phases(code) == 3
    check(p, outs, oracle_run(p, ins))
