"""Integer outputs (Table 1: Cast, Cmp, IsFinite): u8 / i32 tensors written by the virtual machine are compared with
the oracle bit for bit.  Inputs avoid values whose fp32 product lands within rounding distance of an integer, where
the device's fp32 arithmetic and the oracle's float64 may legitimately fall on different sides."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import gpu_run, oracle_run, gate_errors

pytestmark = pytest.mark.gpu


@pytest.fixture(params=[True, False], ids=["lean", "general"])
def interpreter(request):
    dvm.set_lean_kernel(request.param)
    yield request.param
    dvm.set_lean_kernel(True)


def _safe_inputs(shape, dtype, seed, scale):
    """Values x with scale * x at least 1e-3 away from every integer, exactly representable in `dtype`."""
    x = wl.randn(shape, torch.float32, seed) * 3.0
    x = x.to(dtype).to(torch.float32)
    frac = (x * scale) - torch.floor(x * scale)
    bad = (frac < 1e-3) | (frac > 1 - 1e-3)
    x = torch.where(bad, (x + 0.0371).to(dtype).to(torch.float32), x)
    return x.to(dtype)


@pytest.mark.parametrize("shape", [(7, 1531), (33, 1000), (300, 4096), (1, 5), (513, 63)])
@pytest.mark.parametrize("in_dtype", ["f32", "bf16"])
def test_cast_to_i32_and_u8_bit_exact(shape, in_dtype, interpreter):
    prog = wl.program_quantise(in_dtype)
    x = _safe_inputs(shape, torch.bfloat16 if in_dtype == "bf16" else torch.float32, shape[0] + shape[1], 10.0)
    outs, _ = gpu_run(prog, [x])
    want = oracle_run(prog, [x])
    assert outs[0].dtype == torch.int32 and outs[1].dtype == torch.uint8
    assert np.array_equal(outs[0].cpu().numpy().astype(np.float64), want[0])
    assert np.array_equal(outs[1].cpu().numpy().astype(np.float64), want[1])
    g1, _ = gate_errors(wl.to_f64(outs[2]), want[2])
    assert g1 <= 1e-5


def test_cast_saturates_and_maps_nan_to_zero(interpreter):
    prog = wl.program_quantise("f32", 1.0)
    x = torch.tensor([[3e9, -3e9, 300.7, -300.7, float("inf"), float("-inf"), float("nan"), 126.99, -128.5, 0.0]])
    outs, _ = gpu_run(prog, [x])
    want = oracle_run(prog, [x])
    assert np.array_equal(outs[0].cpu().numpy().astype(np.float64), want[0])
    assert np.array_equal(outs[1].cpu().numpy().astype(np.float64), want[1])


@pytest.mark.parametrize("shape", [(3, 50, 333), (2, 7, 4096), (1, 1, 17)])
def test_if_else_add_with_u8_mask(shape):
    """The paper's compound operator with its comparison stored as a byte: the branch taken, bit for bit."""
    prog = wl.program_if_else_add_mask()
    ins = [wl.randn(shape, torch.float32, 50 + i) for i in range(4)]
    outs, _ = gpu_run(prog, ins)
    want = oracle_run(prog, ins)
    assert outs[1].dtype == torch.uint8
    assert np.array_equal(outs[1].cpu().numpy().astype(np.float64), want[1])
    assert set(np.unique(outs[1].cpu().numpy())) <= {0, 1}
    g1, _ = gate_errors(wl.to_f64(outs[0]), want[0])
    assert g1 <= 1e-5


def test_isfinite_and_row_count_as_integers(interpreter):
    """IsFinite stored as u8, and a per-row scalar (the number of positive elements of the row, via Max and Sum)
    stored as i32."""
    p = wl.OpProgram("finite_count")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.unary("isfinite", p.binary("div", a, b)), "u8")
    q = wl.OpProgram("row_count")
    x = q.input("f32", 2)
    pos = q.binary("min", q.binary("max", q.scalar("muls", x, 1e30), x), q.scalar("adds", q.scalar("muls", x, 0.0), 1.0))   # 1 where x > 0 ...
    q.output(q.reduce("sum", q.binary("max", pos, q.scalar("muls", x, 0.0))), "i32")                                       # ... 0 elsewhere
    av = wl.randn((37, 300), torch.float32, 1)
    bv = wl.randn((37, 300), torch.float32, 2)
    bv[::3, ::5] = 0.0
    outs, _ = gpu_run(p, [av, bv])
    assert np.array_equal(outs[0].cpu().numpy().astype(np.float64), oracle_run(p, [av, bv])[0])
    xv = wl.randn((64, 1000), torch.float32, 3)
    outs, _ = gpu_run(q, [xv])
    want = oracle_run(q, [xv])[0]
    assert outs[0].dtype == torch.int32
    assert np.array_equal(outs[0].cpu().numpy().astype(np.float64), want)
    assert np.array_equal(want[:, 0], (xv > 0).sum(dim=1).numpy().astype(np.float64))


def test_integer_inputs_are_rejected():
    p = dvm.Program()
    with pytest.raises(dvm.DvmError):
        p.input("i32", 2)
