"""Edge cases of the interpreter: the longest reducible row, rows one element longer (run in phases), long
non-reduced rows split into column blocks, one-element rows, and the largest stacked launch."""
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


def _layernorm_like():
    p = wl.OpProgram("centre")
    x = p.input("f32", 2)
    mu = p.scalar("muls", p.reduce("sum", x), ("param", 0))
    p.output(p.binary("sub", x, mu), "f32")
    return p


@pytest.mark.parametrize("cols", [8192, 8191, 8189])
def test_longest_reducible_row(cols):
    """256 threads x 32 elements = 8192 columns is the most a reduced row may have (8191 / 8189: misaligned
    rows at full capacity, the last columns wrap around into the head slots)."""
    prog = _layernorm_like()
    x = wl.randn((5, cols), torch.float32, cols)
    outs, code = gpu_run(prog, [x], [1.0 / cols])
    check(prog, outs, oracle_run(prog, [x], [1.0 / cols]))
    assert dvm.code_info(code)["threads_per_row"] == 256


def test_row_longer_than_capacity_runs_in_phases():
    """One column more than a tile holds: the row is walked in column blocks, the mean first, then the difference."""
    prog = _layernorm_like()
    x = wl.randn((3, 8193), torch.float32, 11)
    outs, code = gpu_run(prog, [x], [1.0 / 8193])
    assert "phases    2" in dvm.disassemble(code)
    check(prog, outs, oracle_run(prog, [x], [1.0 / 8193]))


@pytest.mark.parametrize("rows,cols", [(3, 20000), (2, 65537), (1, 100001)])
def test_long_rows_split_into_column_blocks(rows, cols):
    """Without a reduction a row may be any length: it is tiled into column blocks; the row vector operand is
    then loaded per block."""
    p = wl.OpProgram("affine2d")
    x, w, b = p.input("f32", 2), p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("add", p.binary("mul", x, w), b), "f32")
    ins = [wl.randn((rows, cols), torch.float32, 1), wl.randn((1, cols), torch.float32, 2),
           wl.randn((rows, 1), torch.float32, 3)]
    outs, _ = gpu_run(p, ins)
    check(p, outs, oracle_run(p, ins))


@pytest.mark.parametrize("rows", [1, 255, 256, 257, 70000])
def test_one_element_rows(rows):
    """cols = 1: every row is one element (the per-row scalar path on both sides)."""
    p = wl.OpProgram("col")
    x, y = p.input("f32", 2), p.input("f32", 2)
    p.output(p.unary("exp", p.binary("mul", x, y)), "f32")
    ins = [wl.uniform((rows, 1), torch.float32, 4), wl.uniform((rows, 1), torch.float32, 5)]
    outs, _ = gpu_run(p, ins)
    check(p, outs, oracle_run(p, ins))


def test_large_stacked_launch():
    """100 programs in one launch (the programs travel in the 32 KB kernel-parameter block: about 130 of
    this size fit); more than the block holds is refused, not truncated."""
    dvm.set_elems_per_thread(16)
    try:
        prog = wl.program_sigmoid_mul()
        p = dvm.program_from_nodes(prog.nodes)
        codes, tls, meta = [], [], []
        for j in range(100):
            r, c = 1 + (j * 7) % 23, 64 + (j * 37) % 500
            ins, _ = wl.inputs_stack("sigmoid_mul", r, c, 1000 + 3 * j)
            dev = [t.cuda() for t in ins]
            out = torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")
            codes.append(dvm.encode(p, [tuple(t.shape) for t in ins]))
            tls.append(dev + [out])
            meta.append((ins, out))
        dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
        for ins, out in meta:
            check(prog, [out], oracle_run(prog, ins), strict=True)
        with pytest.raises(dvm.DvmError) as ei:
            dvm.launch_stacked(codes * 3, tls * 3)
        assert ei.value.status == -10   # DVM_ERR_TOO_LARGE
    finally:
        dvm.set_elems_per_thread(0)


def test_instance_without_rows_launches_nothing():
    """[0, 300]: a softmax-like program with a reduction encodes (zero tiles), launches nothing and leaves the
    (empty) outputs alone; reducing over an EMPTY axis ([300, 0]) is refused."""
    p = wl.OpProgram("norm")
    x = p.input("f32", 2)
    m = p.reduce("max", x)
    p.output(p.binary("sub", x, m), "f32")
    p.output(m, "f32")
    hp = dvm.program_from_nodes(p.nodes)
    code = dvm.encode(hp, [(0, 300)])
    assert code.out_shapes == [(0, 300), (0, 1)] and dvm.code_info(code)["n_tiles"] == 0
    n0 = dvm.launch_count()
    guard = torch.full((8,), 7.0, device="cuda")
    dvm.launch(code, [guard, guard, guard])
    torch.cuda.synchronize()
    assert dvm.launch_count() == n0 and torch.all(guard == 7.0)
    with pytest.raises(dvm.DvmError) as ei:
        dvm.encode(hp, [(300, 0)])
    assert ei.value.status == -3
