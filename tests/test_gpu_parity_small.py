"""GPU parity: the CUDA virtual machine against the CPU oracle, element by element, on sizes the
oracle finishes in seconds that still span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run, record_strict

pytestmark = pytest.mark.gpu


def _run(prog, inputs, params=(), strict=False):
    outs, code = gpu_run(prog, inputs, params)
    want = oracle_run(prog, inputs, params)
    return check(prog, outs, want, strict=strict), outs, want


def test_c1_exact_config():
    """Config 1: out = exp(a*b + c) - a, fp32 [7, 1531], seed 0."""
    ins = wl.inputs_c1()
    _, outs, want = _run(wl.program_c1(), ins)
    st = record_strict("c1 exp(a*b+c)-a [7,1531]", wl.program_c1(), outs, ins, want_list=want)[0]
    # where fp32 evaluation is well conditioned the device must be right as well: nothing small is zeroed or lost
    assert st["n_well"] > 0.9 * st["n"] and st["well_max"] <= 1e-3


@pytest.mark.parametrize("shape", [(1, 1), (1, 3), (3, 1), (5, 1023), (5, 1024), (5, 1025), (2, 4097),
                                   (37, 4099), (257, 3), (1, 20000), (129, 513)])
def test_c1_shapes(shape):
    ins = [wl.uniform(shape, torch.float32, 100 + i) for i in range(3)]
    _run(wl.program_c1(), ins)


@pytest.mark.parametrize("rows", [1, 2, 3, 255, 256, 257, 1000])
def test_add_rmsnorm(rows):
    """Config 2 program at small row counts: strict gate on both outputs."""
    ins = wl.inputs_add_rmsnorm(rows, 4096, seed=rows)
    (g1, g2), outs, want = _run(wl.program_add_rmsnorm(), ins, strict=True)
    # the updated residual is the exactly rounded sum
    h = (ins[0].double() + ins[1].double()).to(torch.bfloat16)
    assert torch.equal(outs[1].cpu(), h)


@pytest.mark.parametrize("hidden", [8, 64, 100, 1000, 2048, 3072, 4090])
def test_add_rmsnorm_other_widths(hidden):
    ins = wl.inputs_add_rmsnorm(77, hidden, seed=hidden)
    _run(wl.program_add_rmsnorm(hidden=hidden), ins, strict=True)


@pytest.mark.parametrize("B,H,S", [(1, 1, 17), (2, 3, 17), (1, 32, 64), (2, 4, 100), (1, 2, 333), (1, 2, 1000),
                                   (1, 1, 1024), (1, 1, 2047), (1, 1, 2048), (3, 2, 129), (1, 5, 1)])
def test_masked_softmax(B, H, S):
    """Config 3 program: strict gate, masked entries exactly +0, rows sum to 1."""
    ins = wl.inputs_masked_softmax(B, H, S, seed=S)
    _, outs, want = _run(wl.program_masked_softmax(), ins, strict=True)
    o = outs[0].cpu()
    iu = torch.triu_indices(S, S, 1)
    masked = o[..., iu[0], iu[1]]
    assert torch.all(masked == 0) and not torch.any(torch.signbit(masked))
    assert torch.allclose(o.double().sum(-1), torch.ones(B, H, S, dtype=torch.float64), atol=8e-3)


@pytest.mark.parametrize("kind", wl.STACK_KINDS)
@pytest.mark.parametrize("rows,cols", [(1, 64), (3, 65), (512, 64), (7, 777), (33, 1000), (64, 4093),
                                        (5, 4094), (5, 4095), (5, 4096), (300, 2049), (1, 4096)])
def test_stack_kinds_single_launch(kind, rows, cols):
    """Config 4's three programs, each as a single fused instance."""
    ins, params = wl.inputs_stack(kind, rows, cols, seed=rows * 10007 + cols)
    _run(wl.stack_program(kind), ins, params, strict=(kind == "sigmoid_mul"))


def test_fusion_equivalence():
    """Fused add+sqrt equals the chain of single-operator programs, bit for bit (Sec. 5.1)."""
    a = wl.uniform((33, 517), torch.float32, 1, lo=0.0, hi=4.0)
    b = wl.uniform((33, 517), torch.float32, 2, lo=0.0, hi=4.0)
    fused, _ = gpu_run(wl.program_add_sqrt(), [a, b])
    p1 = wl.OpProgram("add"); i0 = p1.input("f32", 2); i1 = p1.input("f32", 2)
    p1.output(p1.binary("add", i0, i1), "f32")
    p2 = wl.OpProgram("sqrt"); j0 = p2.input("f32", 2); p2.output(p2.unary("sqrt", j0), "f32")
    c, _ = gpu_run(p1, [a, b])
    d, _ = gpu_run(p2, [c[0]])
    assert torch.equal(fused[0], d[0])
    # + and sqrt are correctly rounded in fp32, so the result is fixed bit for bit
    ref = torch.sqrt((a + b).double()).float()
    bad = (d[0].cpu() != ref)
    assert not bad.any(), (int(bad.sum()), float((d[0].cpu() - ref).abs().max()),
                           float((torch.sqrt(a + b) - ref).abs().max()))


def test_unaligned_base_pointers():
    """Tensors that start 4 bytes (fp32) / 2 bytes (bf16) into an allocation."""
    prog = wl.program_c1()
    base = [wl.uniform((5 * 1031 + 1,), torch.float32, 7 + i).cuda() for i in range(3)]
    ins = [b[1:].view(5, 1031) for b in base]
    outs, _ = gpu_run(prog, ins)
    check(prog, outs, oracle_run(prog, ins))
    prog = wl.program_add_rmsnorm(hidden=256)
    full = wl.inputs_add_rmsnorm(9, 256, 3)
    xs = torch.empty(9 * 256 + 1, dtype=torch.bfloat16, device="cuda")
    xs[1:] = full[0].flatten().cuda()
    ins = [xs[1:].view(9, 256), full[1].cuda(), full[2].cuda()]
    outs, _ = gpu_run(prog, ins)
    check(prog, outs, oracle_run(prog, ins), strict=True)


def _shifted(t: torch.Tensor, k: int) -> torch.Tensor:
    """A device copy of t that starts k elements into its allocation."""
    buf = torch.empty(t.numel() + k, dtype=t.dtype, device="cuda")
    buf[k:] = t.flatten().cuda()
    return buf[k:].view(t.shape)


@pytest.mark.parametrize("kx,kres,kw,ky", [(1, 0, 0, 0), (3, 3, 0, 0), (5, 2, 7, 0), (0, 1, 0, 3), (7, 7, 7, 7)])
def test_full_capacity_rows_on_misaligned_tensors(kx, kres, kw, ky):
    """Rows of 4096 bf16 fill the whole tile capacity; on a misaligned primary tensor the rows' last columns
    wrap around into the head slots, other operands are realigned, misaligned outputs take the element path."""
    prog = wl.program_add_rmsnorm(4096)
    full = wl.inputs_add_rmsnorm(37, 4096, 5)
    ins = [_shifted(full[0], kx), _shifted(full[1], kres), _shifted(full[2], kw)]
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [tuple(t.shape) for t in ins])
    outs = [_shifted(torch.full((37, 4096), float("nan"), dtype=torch.bfloat16), ky),
            _shifted(torch.full((37, 4096), float("nan"), dtype=torch.bfloat16), 0)]
    dvm.launch(code, ins + outs)
    assert dvm.last_device_status() == 0
    check(prog, outs, oracle_run(prog, full), strict=True)


@pytest.mark.parametrize("cols,k", [(4096, 1), (4095, 0), (4093, 2), (2048, 3), (100, 1)])
def test_layernorm_misaligned_fp32(cols, k):
    """fp32 rows at and next to the full capacity, tensor shifted by k elements."""
    prog = wl.program_layernorm()
    x = wl.randn((19, cols), torch.float32, cols + k)
    xs = _shifted(x, k)
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [(19, cols)], [1.0 / cols])
    out = torch.full((19, cols), float("nan"), dtype=torch.float32, device="cuda")
    dvm.launch(code, [xs, out])
    assert dvm.last_device_status() == 0
    check(prog, [out], oracle_run(prog, [x], [1.0 / cols]))


def test_every_unary_and_binary_op():
    x = wl.uniform((9, 333), torch.float32, 5, lo=0.25, hi=3.0)
    y = wl.uniform((9, 333), torch.float32, 6, lo=0.25, hi=3.0)
    for op in wl.UNARY_OPS:
        p = wl.OpProgram("un_" + op); a = p.input("f32", 2); p.output(p.unary(op, a), "f32")
        xx = x - 1.5 if op in ("abs", "floor", "round", "neg", "erf", "tanh", "sigmoid", "exp") else x
        outs, _ = gpu_run(p, [xx]); check(p, outs, oracle_run(p, [xx]), strict=op not in ("log",))
    for op in wl.BINARY_OPS:
        p = wl.OpProgram("bin_" + op); a = p.input("f32", 2); b = p.input("f32", 2)
        p.output(p.binary(op, a, b), "f32")
        outs, _ = gpu_run(p, [x, y]); check(p, outs, oracle_run(p, [x, y]), strict=op != "sub")
    for op in wl.REDUCE_OPS:
        p = wl.OpProgram("red_" + op); a = p.input("f32", 2); p.output(p.reduce(op, a), "f32")
        outs, _ = gpu_run(p, [x]); check(p, outs, oracle_run(p, [x]), strict=True)


def test_row_scalar_inputs_and_reversed_ops():
    """[R,1] inputs (per-row scalars), scalar-minus-tile and scalar-over-tile forms."""
    p = wl.OpProgram("rowscalar")
    x = p.input("f32", 2); s = p.input("f32", 2); w = p.input("f32", 2)
    t = p.binary("sub", s, x)            # [R,1] - [R,C]
    t = p.binary("div", w, t)            # [1,C] / [R,C]
    r = p.reduce("max", t)
    t = p.binary("sub", r, t)
    p.output(t, "f32"); p.output(r, "f32"); p.output(p.binary("mul", s, s), "f32")
    xs = wl.uniform((41, 300), torch.float32, 1, lo=1.0, hi=2.0)
    ss = wl.uniform((41, 1), torch.float32, 2, lo=3.0, hi=4.0)
    ws = wl.uniform((1, 300), torch.float32, 3, lo=0.5, hi=1.5)
    outs, _ = gpu_run(p, [xs, ss, ws])
    check(p, outs, oracle_run(p, [xs, ss, ws]))


def test_cast_node_and_mixed_dtypes():
    p = wl.OpProgram("mixed")
    x = p.input("f32", 2); y = p.input("bf16", 2)
    t = p.cast(p.binary("mul", x, y), "bf16")
    t = p.scalar("muls", t, 3.0)
    p.output(t, "f32"); p.output(t, "bf16")
    xs = wl.randn((19, 263), torch.float32, 1); ys = wl.randn((19, 263), torch.bfloat16, 2)
    outs, _ = gpu_run(p, [xs, ys])
    want = oracle_run(p, [xs, ys])
    # the cast decides a rounding in fp32 on the device and in fp64 in the oracle: ties can differ by
    # one bf16 ulp, so only the bf16 tolerance applies to this program
    check(p, outs, want, tol=2e-2)


def test_zero_size_and_outputs_untouched():
    prog = wl.program_c1()
    ins = [torch.empty((0, 5), dtype=torch.float32) for _ in range(3)]
    outs, code = gpu_run(prog, ins)
    assert outs[0].shape == (0, 5)
    # a launch writes each output element and nothing else
    a = [wl.uniform((3, 100), torch.float32, i) for i in range(3)]
    import paper_2603_24239_b200 as dvm
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [(3, 100)] * 3)
    buf = torch.full((3 * 100 + 64,), 7.0, dtype=torch.float32, device="cuda")
    out = buf[32:32 + 300].view(3, 100)
    dvm.launch(code, [t.cuda() for t in a] + [out])
    torch.cuda.synchronize()
    assert torch.all(buf[:32] == 7.0) and torch.all(buf[332:] == 7.0)
    check(prog, [out], oracle_run(prog, a))


def test_outer_broadcast_3d():
    """A [1,B,1]-style bias and a [A,1,C] operand: non-mergeable outer dims."""
    p = wl.OpProgram("bcast3")
    x = p.input("f32", 3); b = p.input("f32", 3); c = p.input("f32", 3)
    p.output(p.binary("add", p.binary("mul", x, b), c), "f32")
    xs = wl.randn((5, 7, 130), torch.float32, 1)
    bs = wl.randn((1, 7, 1), torch.float32, 2)
    cs = wl.randn((5, 1, 130), torch.float32, 3)
    outs, _ = gpu_run(p, [xs, bs, cs])
    check(p, outs, oracle_run(p, [xs, bs, cs]))


def _gelu_prog(order=0, scale=1.0 / 2 ** 0.5, reuse_t=False):
    p = wl.OpProgram("gelu_variant")
    x, w = p.input("f32", 2), p.input("f32", 2)
    t = p.binary("mul", x, w)
    u = p.scalar("adds", p.unary("erf", p.scalar("muls", t, scale)), 1.0)
    m = p.binary("mul", t, u) if order == 0 else p.binary("mul", u, t)
    p.output(p.scalar("muls", m, 0.5), "f32")
    if reuse_t:
        p.output(p.scalar("adds", t, 3.0), "f32")
    return p


@pytest.mark.parametrize("order,scale,reuse_t", [(0, 1.0 / 2 ** 0.5, False), (1, 1.0 / 2 ** 0.5, False), (0, 1.0 / 2 ** 0.5, True),
                                                 (0, 0.7, False)])
def test_fused_gelu_matches_the_chain_it_replaces(order, scale, reuse_t):
    """The encoder turns 0.5 * (t * (1 + erf(t / sqrt 2))) into one activation instruction (pattern-based fusion,
    Sec. 5.1); a chain with another constant stays as it is.  Either way the result is the oracle's."""
    prog = _gelu_prog(order, scale, reuse_t)
    ins = [wl.randn((37, 1001), torch.float32, 5), wl.randn((1, 1001), torch.float32, 6)]
    (g1, _), outs, want = _run(prog, ins)
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins])
    assert ("gelu" in dvm.disassemble(code)) == (abs(scale - 1.0 / 2 ** 0.5) < 1e-6)


def test_fused_silu():
    p = wl.OpProgram("silu")
    x, y = p.input("bf16", 2), p.input("bf16", 2)
    p.output(p.binary("mul", p.binary("mul", p.unary("sigmoid", x), x), y), "bf16")
    ins = [wl.randn((129, 513), torch.bfloat16, 1), wl.randn((129, 513), torch.bfloat16, 2)]
    _run(p, ins)
    code = dvm.encode(dvm.program_from_nodes(p.nodes), [tuple(t.shape) for t in ins])
    assert "silu" in dvm.disassemble(code)
