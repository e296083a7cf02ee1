"""GPU parity of Cmp / Select (Table 1) and of the paper's if-else-add compound operator
(a > b ? 2x : 4x) + y.  Comparisons decide a 0/1 value: the device result must equal the oracle's exactly
(both sides compare the same fp32 inputs)."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 1000), (2, 7, 1531), (4, 33, 4096), (1, 2, 8192), (5, 1, 37)])
def test_if_else_add(shape):
    prog = wl.program_if_else_add()
    ins = [wl.randn(shape, torch.float32, 10 + i) for i in range(4)]
    ins[1].view(-1)[::3] = ins[0].view(-1)[::3]          # ties a == b take the else branch
    outs, _ = gpu_run(prog, ins)
    want = oracle_run(prog, ins)
    # 2x, 4x and the add are exact or correctly rounded in fp32: the result is fixed bit for bit
    ref = (torch.where(ins[0] > ins[1], 2 * ins[2], 4 * ins[2]).double() + ins[3].double()).float()
    assert torch.equal(outs[0].cpu(), ref)
    check(prog, outs, want)


@pytest.mark.parametrize("op", wl.COMPARE_OPS)
def test_every_comparison_is_exact(op):
    p = wl.OpProgram("cmp_" + op)
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.compare(op, a, b), "f32")
    x = wl.randn((9, 777), torch.float32, 1)
    y = wl.randn((9, 777), torch.float32, 2)
    y[:, ::5] = x[:, ::5]
    x[0, 0], y[0, 0] = 0.0, -0.0
    outs, _ = gpu_run(p, [x, y])
    want = oracle_run(p, [x, y])[0]
    assert np.array_equal(wl.to_f64(outs[0]), want)


def test_select_forms_and_mixed_dtypes():
    """Condition in the accumulator / then-value in the accumulator / else-value in the accumulator, bf16 and
    fp32 branches, a computed condition that is not 0/1."""
    p = wl.OpProgram("sel")
    c, x, y = p.input("f32", 2), p.input("bf16", 2), p.input("f32", 2)
    s1 = p.select(c, x, y)                                   # condition loaded last: in ACC
    s2 = p.select(c, p.unary("neg", s1), y)                  # then-value in ACC
    s3 = p.select(p.compare("lt", x, y), x, p.scalar("adds", s2, 1.0))   # else-value in ACC
    p.output(s3, "f32")
    p.output(s1, "bf16")
    cc = wl.randn((17, 333), torch.float32, 3)
    cc[cc.abs() < 0.7] = 0.0
    ins = [cc, wl.randn((17, 333), torch.bfloat16, 4), wl.randn((17, 333), torch.float32, 5)]
    outs, code = gpu_run(p, ins)
    check(p, outs, oracle_run(p, ins), strict=True)


def test_compare_on_row_scalars_is_rejected():
    p = wl.OpProgram("cmp_rows")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.compare("gt", a, p.reduce("max", b)), "f32")
    pp = dvm.program_from_nodes(p.nodes)
    with pytest.raises(dvm.DvmError) as ei:
        dvm.encode(pp, [(4, 100), (4, 100)])
    assert ei.value.status == -3


# ---------------------------------------------------------------- Pow, IsFinite (Table 1)
def _rel_err(got, want):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    fin = np.isfinite(want)
    assert np.array_equal(got[~fin & ~np.isnan(want)], want[~fin & ~np.isnan(want)])
    return float(np.max(np.abs(got[fin] - want[fin]) / np.maximum(np.abs(want[fin]), 1e-300))) if fin.any() else 0.0


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(3, 1000), (7, 1531), (2, 5, 4096), (1, 37)])
def test_pow_elementwise(dt, shape):
    """a ^ b with a > 0: every element within 1e-5 (fp32) / 2e-2 (bf16 output) of the oracle, relative."""
    p = wl.OpProgram("pow")
    a, b = p.input(dt, len(shape)), p.input(dt, len(shape))
    p.output(p.binary("pow", a, b), dt)
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    x = (wl.randn(shape, torch.float32, 1).abs() + 0.05).to(tdt)
    y = (wl.randn(shape, torch.float32, 2) * 2).to(tdt)
    outs, code = gpu_run(p, [x, y])
    assert "pow" in dvm.disassemble(code)
    assert _rel_err(wl.to_f64(outs[0]), oracle_run(p, [x, y])[0]) <= (2e-2 if dt == "bf16" else 1e-5)


def test_pow_special_cases_and_mirrored_form():
    """IEEE cases (negative base with integer / non-integer exponent, zero exponents, infinities), and the
    form with the exponent in the accumulator: c ^ (a + b)."""
    p = wl.OpProgram("pow")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("pow", a, b), "f32")
    inf = float("inf")
    x = torch.tensor([[2.0, 2.0, -2.0, -2.0, -2.0, 0.0, 0.0, 5.0, inf, 0.5, 1.0, -1.0]])
    y = torch.tensor([[10.0, -3.0, 3.0, 2.0, 0.5, 0.0, 2.0, 0.0, -1.0, inf, float("nan"), inf]])
    outs, _ = gpu_run(p, [x, y])
    with np.errstate(invalid="ignore"):
        want = oracle_run(p, [x, y])[0]
    assert _rel_err(wl.to_f64(outs[0]), want) <= 1e-6
    q = wl.OpProgram("rpow")
    a, b, c = q.input("f32", 2), q.input("f32", 2), q.input("f32", 2)
    q.output(q.binary("pow", c, q.binary("add", a, b)), "f32")
    ins = [wl.randn((5, 700), torch.float32, 3), wl.randn((5, 700), torch.float32, 4), wl.randn((5, 700), torch.float32, 5).abs() + 0.1]
    outs, code = gpu_run(q, ins)
    assert "rpow" in dvm.disassemble(code)
    assert _rel_err(wl.to_f64(outs[0]), oracle_run(q, ins)[0]) <= 1e-5


def test_isfinite_is_exact_on_tiles_and_on_row_scalars():
    p = wl.OpProgram("isfinite")
    a = p.input("f32", 2)
    p.output(p.unary("isfinite", a), "f32")
    p.output(p.unary("isfinite", p.reduce("sum", a)), "f32")     # one value per row
    x = wl.randn((6, 333), torch.float32, 6)
    x[0, 5], x[1, 7], x[2, 0], x[3, 332] = float("inf"), float("-inf"), float("nan"), 3.0e38
    x[4] = 3.0e38                                                 # the row sum overflows: not finite
    outs, _ = gpu_run(p, [x])
    want = oracle_run(p, [x])
    assert np.array_equal(wl.to_f64(outs[0]), want[0])
    row = wl.to_f64(outs[1]).reshape(-1)
    assert list(row) == [0.0, 0.0, 0.0, 1.0, 0.0, 1.0]           # fp32 row sums: inf, -inf, nan, finite, overflow, finite


def test_if_else_add_many_tiles_single_slot_launch():
    """An instance of thousands of tiles: the program's four fp32 inputs and two temporaries leave room for one
    CTA per SM with two tile slots, so it is encoded for ONE slot per CTA (two CTAs per SM, no prefetch inside a
    CTA).  The result is fixed bit for bit (2x, 4x and the add are exact or correctly rounded)."""
    shape = (61, 67, 4099)
    prog = wl.program_if_else_add()
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [shape] * 4)
    words = np.frombuffer(code.bytes(), dtype=np.uint32)
    assert (int(words[6]) >> 24) & 128          # header word 6 (geometry), flag 128: the single-slot hint
    ins = [wl.randn(shape, torch.float32, 30 + i, "cuda") for i in range(4)]
    out = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
    dvm.launch(code, ins + [out])
    assert dvm.last_device_status() == 0
    ref = (torch.where(ins[0] > ins[1], 2 * ins[2], 4 * ins[2]).double() + ins[3].double()).float()
    assert torch.equal(out, ref)
    rows = [0, 1, 66, 61 * 67 - 1, 1234]
    sub = [t.reshape(-1, shape[2])[rows].cpu() for t in ins]
    want = oracle_run(prog, [s.reshape(1, len(rows), shape[2]) for s in sub])[0]
    got = wl.to_f64(out.reshape(-1, shape[2])[rows])
    assert float(np.max(np.abs(got - want[0]) / np.maximum(np.abs(want[0]), 1e-30))) <= 1e-6   # the oracle does not round to fp32


@pytest.mark.parametrize("kind", ["muls", "adds", "mixed"])
def test_select_between_scalar_multiples_of_one_value(kind):
    """Select(c, x * a, x * b) is encoded as x * Select(c, a, b) (one instruction on the accumulator, no temporaries
    for the candidates; the same with +); candidates of different kinds keep the general form.  Exact either way."""
    p = wl.OpProgram("affine_select")
    a, b, x = p.input("f32", 2), p.input("f32", 2), p.input("f32", 2)
    c = p.compare("le", a, b)
    if kind == "muls":
        u, v = p.scalar("muls", x, 3.0), p.scalar("muls", x, -0.5)
    elif kind == "adds":
        u, v = p.scalar("adds", x, 3.0), p.scalar("adds", x, -0.5)
    else:
        u, v = p.scalar("muls", x, 3.0), p.scalar("adds", x, -0.5)
    p.output(p.select(c, u, v), "f32")
    ins = [wl.randn((37, 1001), torch.float32, 51), wl.randn((37, 1001), torch.float32, 52), wl.randn((37, 1001), torch.float32, 53)]
    outs, code = gpu_run(p, ins)
    text = dvm.disassemble(code)
    assert ("acc ? 3 : -0.5" in text) == (kind != "mixed")
    want = oracle_run(p, ins)
    # one fp32 rounding per element on the device; the oracle's float64 product / sum is exact, rounded here
    assert np.array_equal(wl.to_f64(outs[0]), want[0].astype(np.float32).astype(np.float64))


def test_if_else_add_misaligned_flat_tiles_wrap_around_on_one_slot():
    """fp32 inputs that start 20, 16, 12 and 28 bytes into a 16-byte word, an output 24 bytes in: the flat tiles fill the
    threads' whole capacity, so the first thread's head slots take the tile's last columns (wrap-around; the general
    interpreter, one tile slot per CTA).  The wrapped columns are read one chunk past the thread's last -- and nothing
    further: the last input's image ends the CTA's local memory.  960 tiles, results exact, storage around the
    output untouched."""
    shape, n = (24, 160, 1024), 24 * 160 * 1024
    prog = wl.program_if_else_add()
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [shape] * 4)
    bases = [wl.randn((n + 16,), torch.float32, 90 + i, "cuda") for i in range(4)]
    ins = [b[s:s + n].view(shape) for b, s in zip(bases, (5, 4, 3, 7))]
    obase = torch.full((n + 16,), float("nan"), dtype=torch.float32, device="cuda")
    out = obase[6:6 + n].view(shape)
    dvm.launch(code, ins + [out])
    assert dvm.last_device_status() == 0
    v = dvm.last_launch_variant()
    assert v["lean"] == 0 and v["ctas"] == 3        # wrap-around rows: the general interpreter, its build for one-slot launches
    ref = (torch.where(ins[0] > ins[1], 2 * ins[2], 4 * ins[2]).double() + ins[3].double()).float()
    assert torch.equal(out, ref)
    assert torch.isnan(obase[:6]).all() and torch.isnan(obase[6 + n:]).all()
