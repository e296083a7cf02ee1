"""GPU parity of reductions over another axis than the last (Table 1: Sum / Max / Min of [M, size, N] over
`size` -> [M, 1, N]).  The encoder lowers them to last-axis reductions over permuted views; the oracle reduces
the logical array over the named axis directly."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import TORCH_DT, check, gate_errors, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("op", ["sum", "max", "min"])
@pytest.mark.parametrize("shape,axis", [((3, 50, 7), -2), ((4, 257, 33), -2), ((300, 64), -2), ((5, 6, 70, 9), -3),
                                        ((2, 1000, 1), -2), ((1, 8192, 3), -2), ((6, 40, 8), -3)])
def test_reduce_over_axis(op, shape, axis):
    p = wl.OpProgram("reduce_axis")
    a = p.input("f32", len(shape))
    p.output(p.reduce(op, a, axis), "f32")
    x = wl.randn(shape, torch.float32, len(shape) * 7 - axis)
    outs, code = gpu_run(p, [x])
    want = oracle_run(p, [x])
    exp = list(shape); exp[axis] = 1
    assert list(outs[0].shape) == exp == list(want[0].shape)
    if op == "sum":
        g1, _ = gate_errors(wl.to_f64(outs[0]).reshape(1, -1), want[0].reshape(1, -1))
        assert g1 <= 1e-5
    else:
        assert np.array_equal(wl.to_f64(outs[0]), want[0])      # a max / min picks an input element: exact


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("R,C", [(7, 5), (200, 333), (1024, 64), (4000, 17)])
def test_column_softmax(dt, R, C):
    """softmax over axis -2 of a [R, C] matrix (every column sums to one): two reductions over the row axis and
    tile outputs written back through the permuted view."""
    p = wl.OpProgram("col_softmax")
    x = p.input(dt, 2)
    m = p.reduce("max", x, -2)
    e = p.unary("exp", p.binary("sub", x, m))
    p.output(p.binary("div", e, p.reduce("sum", e, -2)), dt)
    xs = wl.randn((R, C), TORCH_DT[dt], R + C)
    outs, _ = gpu_run(p, [xs])
    want = oracle_run(p, [xs])
    g1, _ = gate_errors(wl.to_f64(outs[0]).T.copy(), want[0].T.copy())     # the reduced axis as the row of the gate
    assert g1 <= (2e-2 if dt == "bf16" else 1e-5), g1
    assert np.allclose(wl.to_f64(outs[0]).sum(axis=0), 1.0, atol=2e-2 if dt == "bf16" else 1e-5)


def test_batchnorm_like_statistics_with_broadcast_operands():
    """y = (x - mean over (S)) * g + b on [B, S, F] with per-feature g, b: mean over axis -2, operands that
    broadcast along the reduced axis, and the statistics as second output."""
    B, S, F = 3, 129, 48
    p = wl.OpProgram("stats")
    x, g, b = p.input("f32", 3), p.input("f32", 1), p.input("f32", 1)
    mean = p.scalar("muls", p.reduce("sum", x, -2), 1.0 / S)
    p.output(p.binary("add", p.binary("mul", p.binary("sub", x, mean), g), b), "f32")
    p.output(mean, "f32")
    ins = [wl.randn((B, S, F), torch.float32, 1), wl.randn((F,), torch.float32, 2), wl.randn((F,), torch.float32, 3)]
    outs, _ = gpu_run(p, ins)
    want = oracle_run(p, ins)
    assert list(outs[1].shape) == [B, 1, F]
    for o, w in zip(outs, want):
        g1, _ = gate_errors(wl.to_f64(o).reshape(1, -1), w.reshape(1, -1))
        assert g1 <= 1e-5


def test_reduce_axis_on_a_view():
    """The lowering composes with caller-given strides: column sums of x[:, 3:40] of a padded buffer."""
    R, C, pitch = 90, 37, 50
    p = wl.OpProgram("colsum")
    a = p.input("f32", 2)
    p.output(p.reduce("sum", a, -2), "f32")
    buf = wl.randn((R * pitch,), torch.float32, 5)
    code = dvm.encode(dvm.program_from_nodes(p.nodes), [(R, C)], in_strides=[[pitch, 1]])
    assert code.out_shapes[0] == (1, C)
    dev = buf.cuda()
    out = torch.full((C,), float("nan"), dtype=torch.float32, device="cuda")
    dvm.launch(code, [dev.data_ptr() + 3 * 4, out])
    assert dvm.last_device_status() == 0
    want = buf.view(R, pitch)[:, 3:3 + C].double().sum(dim=0)
    assert torch.allclose(out.cpu().double(), want, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("op", ["max", "min"])
def test_combined_max_min_signs_and_zeros(op):
    """Results-only max / min over axis -2 go through atomics on the floats' bit patterns: all-negative,
    all-positive, mixed and all-zero columns (with -0.0), many tiles per result element."""
    S, N = 3000, 260
    x = wl.randn((S, N), torch.float32, 77)
    x[:, 0:64] = -x[:, 0:64].abs() - 0.5        # all negative
    x[:, 64:128] = x[:, 64:128].abs() + 0.5     # all positive
    x[:, 128:130] = 0.0
    x[::2, 129] = -0.0
    p = wl.OpProgram("colext")
    a = p.input("f32", 2)
    p.output(p.reduce(op, a, -2), "f32")
    outs, code = gpu_run(p, [x])
    assert "combine=" + op in dvm.disassemble(code)
    want = oracle_run(p, [x])[0]
    assert np.array_equal(wl.to_f64(outs[0]), want)


def test_combined_sum_next_to_a_plain_output():
    """A results-only column sum of squares and the elementwise result itself, from one program."""
    M, S, N = 3, 700, 96
    p = wl.OpProgram("sq_and_colsum")
    a = p.input("bf16", 3)
    sq = p.binary("mul", a, a)
    p.output(sq, "bf16")
    p.output(p.reduce("sum", sq, -2), "f32")
    x = wl.randn((M, S, N), torch.bfloat16, 5)
    outs, code = gpu_run(p, [x])
    assert "combine=sum" in dvm.disassemble(code)
    want = oracle_run(p, [x])
    g1, _ = gate_errors(wl.to_f64(outs[0]).reshape(1, -1), want[0].reshape(1, -1))
    assert g1 <= 2e-2
    g1, _ = gate_errors(wl.to_f64(outs[1]).reshape(1, -1), want[1].reshape(1, -1))
    assert g1 <= 1e-5
