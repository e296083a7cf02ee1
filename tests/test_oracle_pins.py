"""Pins for the CPU oracle: things the paper and the mathematics fix, none of
which is the oracle's own formula retyped.

 * a scalar, pure-Python evaluator (math module, explicit broadcast indexing)
   as brute force on tiny inputs;
 * closed forms of each benchmark program;
 * torch float64 library routines on the special cases they cover;
 * hand-computed bf16 rounding cases.
"""
import math

import numpy as np
import pytest
import torch

import dvm_workloads as wl
from oracle import dvm_oracle as orc

RNG = np.random.default_rng(12345)


# ---------------------------------------------------------------- brute force
def _bcast_index(idx, shape, out_rank):
    """Index into an array of `shape` for output index `idx` (right-aligned)."""
    pad = out_rank - len(shape)
    return tuple(0 if shape[d] == 1 else idx[pad + d] for d in range(len(shape)))


def brute(nodes, inputs, params=()):
    """Element-by-element evaluation with Python floats.  Tiny inputs only."""
    un = {"exp": math.exp, "sqrt": math.sqrt, "abs": abs, "log": math.log,
          "floor": math.floor, "erf": math.erf, "neg": lambda v: -v,
          "rsqrt": lambda v: 1.0 / math.sqrt(v), "recip": lambda v: 1.0 / v,
          "sigmoid": lambda v: 1.0 / (1.0 + math.exp(-v)), "tanh": math.tanh,
          "round": lambda v: float(round(v)),   # Python round() is half-to-even
          "isfinite": lambda v: 1.0 if math.isfinite(v) else 0.0}
    bi = {"add": lambda a, b: a + b, "sub": lambda a, b: a - b, "mul": lambda a, b: a * b,
          "div": lambda a, b: a / b, "max": max, "min": min, "pow": math.pow}
    vals, shapes, outs = {}, {}, []
    it = iter(inputs)
    for i, n in enumerate(nodes):
        k = n[0]
        if k == "input":
            a = np.asarray(next(it), dtype=np.float64)
            shapes[i] = a.shape
            vals[i] = {idx: float(a[idx]) for idx in np.ndindex(a.shape)}
        elif k in ("unary", "scalar", "cast"):
            src = n[2] if k != "cast" else n[1]
            shapes[i] = shapes[src]
            if k == "unary":
                f = un[n[1]]
            elif k == "scalar":
                s = n[3]
                s = float(np.float32(params[s[1]] if isinstance(s, tuple) else s))
                f = (lambda v, s=s: v + s) if n[1] == "adds" else (lambda v, s=s: v * s)
            else:
                tdt = torch.bfloat16 if n[2] == "bf16" else torch.float32
                f = lambda v, tdt=tdt: float(torch.tensor(v, dtype=torch.float64).to(tdt))
            vals[i] = {idx: f(v) for idx, v in vals[src].items()}
        elif k == "binary":
            sa, sb = shapes[n[2]], shapes[n[3]]
            r = max(len(sa), len(sb))
            pa, pb = (1,) * (r - len(sa)) + sa, (1,) * (r - len(sb)) + sb
            so = tuple(max(x, y) for x, y in zip(pa, pb))
            shapes[i] = so
            vals[i] = {idx: bi[n[1]](vals[n[2]][_bcast_index(idx, sa, r)],
                                     vals[n[3]][_bcast_index(idx, sb, r)])
                       for idx in np.ndindex(so)}
        elif k == "reduce":
            s = shapes[n[2]]
            ax = len(s) + (n[3] if len(n) > 3 else -1)
            so = s[:ax] + (1,) + s[ax + 1:]
            shapes[i] = so
            red = {"sum": sum, "max": max, "min": min}[n[1]]
            vals[i] = {idx: red(vals[n[2]][idx[:ax] + (j,) + idx[ax + 1:]] for j in range(s[ax]))
                       for idx in np.ndindex(so)}
        elif k == "matmul":
            (M, K), (K2, N) = shapes[n[1]], shapes[n[2]]
            assert K == K2
            shapes[i] = (M, N)
            vals[i] = {(r, c): sum(vals[n[1]][(r, kk)] * vals[n[2]][(kk, c)] for kk in range(K))
                       for r in range(M) for c in range(N)}
        elif k == "output":
            o = np.empty(shapes[n[1]])
            for idx, v in vals[n[1]].items():
                o[idx] = v
            outs.append(o)
    return outs


def _tiny_inputs(prog, shapes):
    ins = []
    for s in shapes:
        ins.append(RNG.normal(size=s))
    return ins


TINY = [
    (wl.program_c1(), [(3, 5)] * 3, ()),
    (wl.program_add_rmsnorm(hidden=6), [(4, 6), (4, 6), (6,)], ()),
    (wl.program_masked_softmax(), [(2, 3, 4, 4), (1, 1, 4, 4)], ()),
    (wl.program_gelu_affine(), [(3, 7), (1, 7), (1, 7)], ()),
    (wl.program_layernorm(), [(3, 9)], (1.0 / 9,)),
    (wl.program_sigmoid_mul(), [(2, 5), (2, 5)], ()),
    (wl.program_mlp_gate(), [(3, 4), (4, 5), (4, 5)], ()),
    (wl.program_add_sqrt(), [(2, 3), (2, 3)], ()),
]


@pytest.mark.parametrize("prog,shapes,params", TINY, ids=[t[0].name for t in TINY])
def test_matches_scalar_brute_force(prog, shapes, params):
    ins = _tiny_inputs(prog, shapes)
    if prog.name == "add_sqrt":
        ins = [np.abs(a) for a in ins]
    got = orc.evaluate(prog.nodes, ins, params)
    want = brute(prog.nodes, ins, params)
    assert len(got) == len(want)
    for g, w in zip(got, want):
        assert g.shape == w.shape
        np.testing.assert_allclose(g, w, rtol=1e-13, atol=1e-15)


def test_every_primitive_against_brute_force():
    x = RNG.uniform(0.1, 3.0, size=(2, 5))
    y = RNG.uniform(0.1, 3.0, size=(1, 5))
    for op in wl.UNARY_OPS:
        p = wl.OpProgram()
        a = p.input("f32", 2)
        p.output(p.unary(op, a), "f32")
        xx = x - 1.5 if op in ("abs", "floor", "round", "neg", "erf", "tanh", "sigmoid", "exp") else x
        np.testing.assert_allclose(orc.evaluate(p.nodes, [xx])[0], brute(p.nodes, [xx])[0], rtol=1e-14)
    for op in wl.BINARY_OPS:
        p = wl.OpProgram()
        a, b = p.input("f32", 2), p.input("f32", 2)
        p.output(p.binary(op, a, b), "f32")
        xa = x if op == "pow" else x - 1   # math.pow raises on a negative base with a non-integer exponent
        np.testing.assert_allclose(orc.evaluate(p.nodes, [xa, y - 1])[0],
                                   brute(p.nodes, [xa, y - 1])[0], rtol=1e-14)
    for op in wl.REDUCE_OPS:
        p = wl.OpProgram()
        a = p.input("f32", 2)
        p.output(p.reduce(op, a), "f32")
        np.testing.assert_allclose(orc.evaluate(p.nodes, [x])[0], brute(p.nodes, [x])[0], rtol=1e-14)


# ---------------------------------------------------------------- primitives: exact identities
def test_primitive_identities():
    def run1(kind, op, x, *extra):
        p = wl.OpProgram()
        a = p.input("f32", 1)
        v = getattr(p, kind)(op, a, *extra)
        p.output(v, "f32")
        return orc.evaluate(p.nodes, [np.asarray(x, dtype=np.float64)])[0]

    assert run1("unary", "exp", [0.0])[0] == 1.0
    assert run1("unary", "sqrt", [4.0])[0] == 2.0
    assert run1("unary", "log", [1.0])[0] == 0.0
    assert run1("unary", "abs", [-3.5])[0] == 3.5
    assert run1("unary", "rsqrt", [0.25])[0] == 2.0
    assert run1("unary", "recip", [8.0])[0] == 0.125
    assert run1("unary", "sigmoid", [0.0])[0] == 0.5
    assert run1("unary", "erf", [0.0])[0] == 0.0
    assert list(run1("unary", "floor", [-1.5, 1.5])) == [-2.0, 1.0]
    assert list(run1("unary", "round", [0.5, 1.5, 2.5, -0.5])) == [0.0, 2.0, 2.0, -0.0]
    assert run1("scalar", "adds", [1.0], 0.5)[0] == 1.5
    assert run1("scalar", "muls", [3.0], 0.5)[0] == 1.5
    # Adds/Muls equal Add/Mul with a broadcast scalar tensor
    x = RNG.normal(size=(4, 3))
    p = wl.OpProgram(); a = p.input("f32", 2); p.output(p.scalar("muls", a, 0.375), "f32")
    q = wl.OpProgram(); a = q.input("f32", 2); s = q.input("f32", 2); q.output(q.binary("mul", a, s), "f32")
    np.testing.assert_array_equal(orc.evaluate(p.nodes, [x])[0],
                                  orc.evaluate(q.nodes, [x, np.full((1, 1), 0.375)])[0])


def test_scalar_immediate_is_fp32():
    p = wl.OpProgram(); a = p.input("f32", 1); p.output(p.scalar("muls", a, 0.1), "f32")
    got = orc.evaluate(p.nodes, [np.array([1.0])])[0][0]
    assert got == float(np.float32(0.1)) and got != 0.1


def test_sub_div_operand_order():
    p = wl.OpProgram(); a = p.input("f32", 1); b = p.input("f32", 1)
    p.output(p.binary("sub", a, b), "f32"); p.output(p.binary("div", a, b), "f32")
    s, d = orc.evaluate(p.nodes, [np.array([6.0]), np.array([2.0])])
    assert s[0] == 4.0 and d[0] == 3.0


# ---------------------------------------------------------------- rounding
def test_bf16_rounding_hand_cases():
    e = 2.0 ** -8          # half of the bf16 spacing at 1.0 (2^-7)
    cases = {
        1.0: 1.0,
        1.0 + e: 1.0,                          # tie -> even (mantissa 0)
        1.0 + 3 * e: 1.0 + 4 * e,              # tie -> even (mantissa 2)
        1.0 + e + 2.0 ** -40: 1.0 + 2 * e,     # above the tie only in float64: double rounding trap
        1.0 + e - 2.0 ** -40: 1.0,
        -(1.0 + e + 2.0 ** -40): -(1.0 + 2 * e),
        3.140625: 3.140625,                    # exactly representable
        0.0: 0.0,
    }
    got = orc.round_to_bf16(np.array(list(cases.keys())))
    np.testing.assert_array_equal(got, np.array(list(cases.values())))
    assert np.isnan(orc.round_to_bf16(np.array([np.nan])))[0]
    assert orc.round_to_bf16(np.array([-np.inf]))[0] == -np.inf


def test_bf16_rounding_matches_torch_on_fp32_values():
    x32 = torch.randn(20000, generator=torch.Generator().manual_seed(5)) * 37.0
    want = x32.to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.round_to_bf16(x32.to(torch.float64).numpy())
    np.testing.assert_array_equal(got, want)


def test_cast_node_rounds():
    p = wl.OpProgram(); a = p.input("f32", 1)
    p.output(p.cast(a, "bf16"), "f32"); p.output(p.cast(a, "f32"), "f32")
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 2.0 ** -30])
    b, f = orc.evaluate(p.nodes, [x])
    assert list(b) == [1.0 + 2.0 ** -7, 1.0]
    assert list(f) == [float(np.float32(x[0])), 1.0]


# ---------------------------------------------------------------- broadcasting
def test_broadcast_equals_materialised():
    p = wl.program_gelu_affine()
    x, w, b = RNG.normal(size=(5, 8)), RNG.normal(size=(1, 8)), RNG.normal(size=(1, 8))
    a = orc.evaluate(p.nodes, [x, w, b])[0]
    c = orc.evaluate(p.nodes, [x, np.repeat(w, 5, 0), np.repeat(b, 5, 0)])[0]
    np.testing.assert_array_equal(a, c)
    # w = 1, b = 0 reduces the affine part to x: GELU(x) against torch
    g = orc.evaluate(p.nodes, [x, np.ones((1, 8)), np.zeros((1, 8))])[0]
    want = torch.nn.functional.gelu(torch.tensor(x, dtype=torch.float64)).numpy()
    # 1/sqrt(2) enters as an fp32 immediate: relative error of the argument 3e-8
    np.testing.assert_allclose(g, want, rtol=1e-6, atol=1e-8)

    q = wl.program_masked_softmax()
    s = RNG.normal(size=(2, 3, 6, 6))
    m = wl.to_f64(wl.causal_mask(6))
    a = orc.evaluate(q.nodes, [s, m])[0]
    c = orc.evaluate(q.nodes, [s, np.broadcast_to(m, s.shape).copy()])[0]
    np.testing.assert_array_equal(a, c)


# ---------------------------------------------------------------- C1
def test_c1_closed_forms():
    p = wl.program_c1()
    a, b, c = (wl.to_f64(t) for t in wl.inputs_c1())
    out = orc.evaluate(p.nodes, [a, b, c])[0]
    np.testing.assert_allclose(out, np.exp(a * b + c) - a, rtol=1e-15)
    z = np.zeros_like(a)
    np.testing.assert_array_equal(orc.evaluate(p.nodes, [a, z, z])[0], 1.0 - a)
    np.testing.assert_array_equal(orc.evaluate(p.nodes, [z, b, c])[0], np.exp(c))


# ---------------------------------------------------------------- softmax
def test_softmax_closed_forms():
    p = wl.program_masked_softmax()
    B, H, S = 2, 3, 19
    s, m = (wl.to_f64(t) for t in wl.inputs_masked_softmax(B, H, S, 11))
    out = orc.evaluate(p.nodes, [s, m])[0]
    assert out.shape == (B, H, S, S)
    np.testing.assert_allclose(out.sum(-1), 1.0, rtol=0, atol=1e-14)       # rows sum to 1
    assert np.all(out[..., 0, 0] == 1.0) and np.all(out[..., 0, 1:] == 0)    # causal row 0
    iu = np.triu_indices(S, 1)
    assert np.all(out[..., iu[0], iu[1]] == 0.0)                             # masked exactly +0
    assert not np.any(np.signbit(out))
    # equal scores: row i is 1/(i+1) on j <= i
    eq = orc.evaluate(p.nodes, [np.full((1, 1, S, S), 0.75), m])[0][0, 0]
    for i in range(S):
        np.testing.assert_allclose(eq[i, :i + 1], 1.0 / (i + 1), rtol=1e-15)
    # shift invariance
    sh = orc.evaluate(p.nodes, [s + 3.0, m])[0]
    np.testing.assert_allclose(sh, out, rtol=1e-12, atol=1e-18)
    # library routine
    scale = float(np.float32(1.0 / math.sqrt(128)))
    want = torch.softmax((torch.tensor(s) + torch.tensor(m)) * scale, dim=-1).numpy()
    np.testing.assert_allclose(out, want, rtol=1e-13, atol=1e-18)
    # mask-then-scale equals scale-then-mask for a 0/-inf mask
    alt = torch.softmax(torch.tensor(s) * scale + torch.tensor(m), dim=-1).numpy()
    np.testing.assert_allclose(out, alt, rtol=1e-13, atol=1e-18)


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_closed_forms():
    Hd = 64
    p = wl.program_add_rmsnorm(hidden=Hd, eps=1e-6)
    x, res, w = (wl.to_f64(t) for t in wl.inputs_add_rmsnorm(9, Hd, 3))
    y, h = orc.evaluate(p.nodes, [x, res, w])
    np.testing.assert_array_equal(h, x + res)                         # residual stream is exact
    ones = np.ones(Hd)
    y1, _ = orc.evaluate(p.nodes, [x, res, ones])
    ms = np.mean((x + res) ** 2, axis=-1)
    np.testing.assert_allclose(np.sqrt(np.mean(y1 ** 2, -1)), np.sqrt(ms / (ms + 1e-6)), rtol=1e-9)
    np.testing.assert_allclose(np.sqrt(np.mean(y1 ** 2, -1)), 1.0, atol=5e-6)   # unit RMS
    np.testing.assert_allclose(y, y1 * w, rtol=1e-15)                 # weight applies elementwise
    # constant row c -> c / sqrt(c^2 + eps)
    c = 0.5
    yc, _ = orc.evaluate(p.nodes, [np.full((1, Hd), c), np.zeros((1, Hd)), ones])
    np.testing.assert_allclose(yc, c / math.sqrt(c * c + float(np.float32(1e-6))), rtol=1e-9)
    # positive scale invariance up to eps
    y4, _ = orc.evaluate(p.nodes, [4 * x, 4 * res, ones])
    np.testing.assert_allclose(y4, y1, rtol=1e-5)
    # library routine
    want = torch.nn.functional.rms_norm(torch.tensor(x + res), (Hd,), torch.tensor(w),
                                        eps=float(np.float32(1e-6))).numpy()
    np.testing.assert_allclose(y, want, rtol=1e-9)


# ---------------------------------------------------------------- LayerNorm
def test_layernorm_closed_forms():
    p = wl.program_layernorm()
    cols = 37
    x = RNG.normal(size=(6, cols)) * 3 + 1
    (o,) = orc.evaluate(p.nodes, [x], (1.0 / cols,))
    v = x.var(-1)
    np.testing.assert_allclose(o.mean(-1), 0.0, atol=1e-7)   # 1/37 is an fp32 immediate
    np.testing.assert_allclose(o.var(-1), v / (v + 1e-5), rtol=1e-6)
    want = torch.nn.functional.layer_norm(torch.tensor(x), (cols,), eps=1e-5).numpy()
    np.testing.assert_allclose(o, want, rtol=1e-6, atol=1e-7)   # 1/cols is an fp32 immediate
    # exact-in-fp32 reciprocal: cols = 32
    x32 = RNG.normal(size=(4, 32))
    (o32,) = orc.evaluate(p.nodes, [x32], (1.0 / 32,))
    want = torch.nn.functional.layer_norm(torch.tensor(x32), (32,), eps=float(np.float32(1e-5))).numpy()
    np.testing.assert_allclose(o32, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(o32.mean(-1), 0.0, atol=1e-15)
    (oc,) = orc.evaluate(p.nodes, [np.full((1, 32), 2.5)], (1.0 / 32,))
    assert np.all(oc == 0.0)                                         # constant row -> 0
    alt = np.tile([1.0, -1.0], 16)[None]
    (oa,) = orc.evaluate(p.nodes, [alt], (1.0 / 32,))
    np.testing.assert_allclose(oa, alt / math.sqrt(1 + float(np.float32(1e-5))), rtol=1e-14)


# ---------------------------------------------------------------- GELU / sigmoid / SiLU
def test_gelu_sigmoid_identities():
    p = wl.program_gelu_affine()
    t = RNG.normal(size=(3, 10)) * 2
    one, zero = np.ones((1, 10)), np.zeros((1, 10))
    g_pos = orc.evaluate(p.nodes, [t, one, zero])[0]
    g_neg = orc.evaluate(p.nodes, [-t, one, zero])[0]
    np.testing.assert_allclose(g_pos - g_neg, t, rtol=1e-6, atol=1e-7)   # 1/sqrt(2) is fp32
    assert orc.evaluate(p.nodes, [np.zeros((1, 10)), one, zero])[0].max() == 0.0

    q = wl.program_sigmoid_mul()
    x, y = RNG.normal(size=(4, 6)) * 4, RNG.normal(size=(4, 6))
    o = orc.evaluate(q.nodes, [x, y])[0]
    on = orc.evaluate(q.nodes, [-x, y])[0]
    np.testing.assert_allclose(o + on, y, rtol=1e-13)                    # s(x) + s(-x) = 1
    np.testing.assert_array_equal(orc.evaluate(q.nodes, [np.zeros((4, 6)), y])[0], y / 2)
    np.testing.assert_allclose(o, (torch.sigmoid(torch.tensor(x)) * torch.tensor(y)).numpy(), rtol=1e-13)


# ---------------------------------------------------------------- matmul + epilogue
def test_mlp_gate_closed_forms():
    p = wl.program_mlp_gate()
    K, N = 8, 5
    wg, wu = RNG.normal(size=(K, N)), RNG.normal(size=(K, N))
    # X = I picks out the weight rows
    o = orc.evaluate(p.nodes, [np.eye(K), wg, wu])[0]
    np.testing.assert_allclose(o, wg / (1 + np.exp(-wg)) * wu, rtol=1e-14)
    # W_gate = 0 -> 0
    x = RNG.normal(size=(3, K))
    assert np.all(orc.evaluate(p.nodes, [x, np.zeros((K, N)), wu])[0] == 0)
    # all ones -> K * sigmoid(K) * K
    o1 = orc.evaluate(p.nodes, [np.ones((2, K)), np.ones((K, N)), np.ones((K, N))])[0]
    np.testing.assert_allclose(o1, K / (1 + math.exp(-K)) * K, rtol=1e-14)
    # non-square, transposition-sensitive: triple loop
    M = 4
    g = np.zeros((M, N)); u = np.zeros((M, N))
    xx = RNG.normal(size=(M, K))
    for i in range(M):
        for j in range(N):
            for k in range(K):
                g[i, j] += xx[i, k] * wg[k, j]
                u[i, j] += xx[i, k] * wu[k, j]
    want = torch.nn.functional.silu(torch.tensor(g)).numpy() * u
    np.testing.assert_allclose(orc.evaluate(p.nodes, [xx, wg, wu])[0], want, rtol=1e-12)


# ---------------------------------------------------------------- fusion equivalence (Sec. 5.1)
def test_fused_equals_chain_of_single_ops():
    a, b = np.abs(RNG.normal(size=(3, 4))), np.abs(RNG.normal(size=(3, 4)))
    fused = orc.evaluate(wl.program_add_sqrt().nodes, [a, b])[0]
    p1 = wl.OpProgram(); i0 = p1.input("f32", 2); i1 = p1.input("f32", 2); p1.output(p1.binary("add", i0, i1), "f32")
    p2 = wl.OpProgram(); i0 = p2.input("f32", 2); p2.output(p2.unary("sqrt", i0), "f32")
    c = orc.evaluate(p1.nodes, [a, b])[0]
    np.testing.assert_array_equal(fused, orc.evaluate(p2.nodes, [c])[0])


def test_oracle_does_not_import_product():
    import ast, os
    src = open(os.path.join(os.path.dirname(orc.__file__), "dvm_oracle.py")).read()
    mods = set()
    for node in ast.walk(ast.parse(src)):
        if isinstance(node, ast.Import):
            mods |= {a.name.split(".")[0] for a in node.names}
        elif isinstance(node, ast.ImportFrom):
            mods.add((node.module or "").split(".")[0])
    assert mods <= {"__future__", "numpy", "scipy"}, mods


# ---------------------------------------------------------------- compare / select
def test_compare_and_select_definitions():
    """Cmp gives 1 where the relation holds; Select takes x where cond != 0 (Table 1).  Pinned by hand values,
    by the complement identities gt + le = 1 / eq + ne = 1, and by max(a, b) = select(a > b, a, b)."""
    a = np.array([[1.0, 2.0, 3.0, -0.0], [5.0, -1.0, 2.5, 0.0]])
    b = np.array([[1.0, 3.0, 2.0, 0.0], [4.0, -1.0, 2.5, -7.0]])
    def run(build):
        p = wl.OpProgram("t"); x, y = p.input("f32", 2), p.input("f32", 2); p.output(build(p, x, y), "f32")
        return orc.evaluate(p.nodes, [a, b])[0]
    assert np.array_equal(run(lambda p, x, y: p.compare("gt", x, y)), [[0, 0, 1, 0], [1, 0, 0, 1]])
    assert np.array_equal(run(lambda p, x, y: p.compare("eq", x, y)), [[1, 0, 0, 1], [0, 1, 1, 0]])   # -0 == +0
    for u, v in (("gt", "le"), ("ge", "lt"), ("eq", "ne")):
        assert np.array_equal(run(lambda p, x, y: p.compare(u, x, y)) + run(lambda p, x, y: p.compare(v, x, y)), np.ones((2, 4)))
    assert np.array_equal(run(lambda p, x, y: p.select(p.compare("gt", x, y), x, y)), np.maximum(a, b))
    assert np.array_equal(run(lambda p, x, y: p.select(p.compare("lt", x, y), x, y)), np.minimum(a, b))
    # a non-0/1 condition value counts as true
    assert np.array_equal(run(lambda p, x, y: p.select(y, x, y)), np.where(b != 0, a, b))


def test_if_else_add_closed_form():
    """(a > b ? 2x : 4x) + y against the formula written out with numpy; a == b takes the else branch."""
    rng = np.random.default_rng(3)
    a, b, x, y = (rng.standard_normal((3, 5, 7)) for _ in range(4))
    b[0, 0, :3] = a[0, 0, :3]
    got = orc.evaluate(wl.program_if_else_add().nodes, [a, b, x, y])[0]
    want = np.where(a > b, 2.0 * x, 4.0 * x) + y
    assert np.array_equal(got, want)
    assert np.array_equal(got[0, 0, :3], 4.0 * x[0, 0, :3] + y[0, 0, :3])


# ---------------------------------------------------------------- views (Table 1, ViewLoad / ViewStore)
def test_view_load_against_library_views_and_brute_force():
    """view_load is pinned by numpy's own transposes, slices and broadcasts (another mechanism: numpy's
    stride machinery) and by an explicit loop over index tuples on a tiny case."""
    base = RNG.standard_normal((4, 6, 10))
    flat = base.reshape(-1)
    es = base.itemsize
    for v in (base.transpose(1, 0, 2), base[:, 1:5, 2:9], base[::2, :, ::3], base.transpose(2, 0, 1)[3:, 1:],
              np.broadcast_to(base[:, :1, :], (4, 6, 10)), base[1]):
        off = (v.__array_interface__["data"][0] - base.__array_interface__["data"][0]) // es
        got = orc.view_load(flat, off, v.shape, [t // es for t in v.strides])
        assert np.array_equal(got, v)
    shape, strides, off = (2, 3, 2), (7, 2, 30), 5
    got = orc.view_load(flat, off, shape, strides)
    for i in range(2):
        for j in range(3):
            for k in range(2):
                assert got[i, j, k] == flat[off + 7 * i + 2 * j + 30 * k]
    with pytest.raises(IndexError):
        orc.view_load(flat, 0, (5, 100), (60, 1))


def test_view_store_writes_the_view_and_nothing_else():
    storage = np.arange(240, dtype=np.float64).reshape(4, 60)
    vals = -1.0 - RNG.random((3, 5, 2))
    out = orc.view_store(storage, 7, (3, 5, 2), (60, 4, 1), vals)
    want = storage.copy().reshape(-1)
    for i in range(3):
        for j in range(5):
            for k in range(2):
                want[7 + 60 * i + 4 * j + k] = vals[i, j, k]
    assert np.array_equal(out.reshape(-1), want) and out.shape == storage.shape
    assert np.array_equal(storage, np.arange(240, dtype=np.float64).reshape(4, 60))  # the input is not modified
    assert np.array_equal(orc.view_load(out, 7, (3, 5, 2), (60, 4, 1)), vals)       # load after store returns the values
    with pytest.raises(ValueError):
        orc.view_store(storage, 0, (3, 4), (2, 1), np.zeros((3, 4)))                # rows overlap: aliasing


# ---------------------------------------------------------------- Pow, IsFinite (Table 1)
def test_pow_against_math_pow_and_closed_forms():
    """Pow is pinned by the C library's pow through math.pow, element by element, and by the identities
    x^2 = x*x, x^0.5 = sqrt(x), x^0 = 1, x^-1 = 1/x, 2^k exact."""
    p = wl.OpProgram("pow")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("pow", a, b), "f32")
    x = np.abs(RNG.standard_normal((5, 7))) + 0.1
    y = RNG.standard_normal((5, 7)) * 3
    got = orc.evaluate(p.nodes, [x, y])[0]
    for i in range(5):
        for j in range(7):
            assert got[i, j] == pytest.approx(math.pow(x[i, j], y[i, j]), rel=1e-15)
    ev = lambda xx, yy: orc.evaluate(p.nodes, [np.asarray(xx, dtype=np.float64).reshape(1, -1), np.asarray(yy, dtype=np.float64).reshape(1, -1)])[0][0]
    assert np.allclose(ev(x[0], np.full(7, 2.0)), x[0] * x[0], rtol=1e-15)
    assert np.allclose(ev(x[0], np.full(7, 0.5)), np.sqrt(x[0]), rtol=1e-15)
    assert np.array_equal(ev(x[0], np.zeros(7)), np.ones(7))
    assert np.allclose(ev(x[0], np.full(7, -1.0)), 1.0 / x[0], rtol=1e-15)
    assert np.array_equal(ev([2.0, 2.0, 2.0, -2.0, -2.0], [10.0, -3.0, 0.0, 3.0, 2.0]), [1024.0, 0.125, 1.0, -8.0, 4.0])
    with np.errstate(invalid="ignore"):
        assert np.isnan(ev([-2.0], [0.5])[0])          # negative base, non-integer exponent


def test_isfinite_flags():
    p = wl.OpProgram("isfinite")
    a = p.input("f32", 2)
    p.output(p.unary("isfinite", a), "f32")
    x = np.array([[0.0, -0.0, 1.5, -3e38, np.inf, -np.inf, np.nan, 1e-45]])
    got = orc.evaluate(p.nodes, [x])[0]
    assert np.array_equal(got, [[1, 1, 1, 1, 0, 0, 0, 1]])
    assert np.array_equal(got[0], [1.0 if math.isfinite(v) else 0.0 for v in x[0]])


# ---------------------------------------------------------------- reductions over another axis (Table 1, [M,size,N] -> [M,1,N])
def test_reduce_over_the_penultimate_and_outer_axes():
    """Pinned by closed forms (sums of index patterns), by the last-axis reduction of the swapped array
    (numpy's swapaxes: another mechanism) and by brute force over index tuples."""
    M, S, N = 3, 5, 4
    x = RNG.standard_normal((M, S, N))
    for op, ref in (("sum", np.sum), ("max", np.max), ("min", np.min)):
        for axis in (-1, -2, -3):
            p = wl.OpProgram()
            a = p.input("f32", 3)
            p.output(p.reduce(op, a, axis), "f32")
            got = orc.evaluate(p.nodes, [x])[0]
            want_shape = list(x.shape); want_shape[axis] = 1
            assert list(got.shape) == want_shape
            swapped = ref(np.swapaxes(x, axis, -1), axis=-1, keepdims=True)
            assert np.array_equal(got, np.swapaxes(swapped, axis, -1))
            np.testing.assert_allclose(got, brute(p.nodes, [x])[0], rtol=1e-14)
    # closed form: x[m, s, n] = 100 m + 10 s + n  ->  sum over s = S (100 m + n) + 10 S (S - 1) / 2, max over s at s = S - 1
    idx = np.indices((M, S, N)).astype(np.float64)
    y = 100 * idx[0] + 10 * idx[1] + idx[2]
    p = wl.OpProgram()
    a = p.input("f32", 3)
    p.output(p.reduce("sum", a, -2), "f32")
    p.output(p.reduce("max", a, -2), "f32")
    s_, m_ = orc.evaluate(p.nodes, [y])
    mm, nn = np.meshgrid(np.arange(M), np.arange(N), indexing="ij")
    assert np.array_equal(s_[:, 0, :], S * (100 * mm + nn) + 10 * S * (S - 1) / 2)
    assert np.array_equal(m_[:, 0, :], 100 * mm + 10 * (S - 1) + nn)
    # a column normalisation: x / sum over rows; every column of the result sums to 1
    q = wl.OpProgram()
    a = q.input("f32", 2)
    q.output(q.binary("div", a, q.reduce("sum", a, -2)), "f32")
    z = np.abs(RNG.standard_normal((7, 6))) + 0.1
    assert np.allclose(orc.evaluate(q.nodes, [z])[0].sum(axis=0), 1.0, rtol=1e-14)


# ---------------------------------------------------------------- integer types (Table 1: Cast, Cmp, IsFinite)
def test_cast_to_int_drops_the_fraction_toward_zero():
    """Hand table, and numpy's own trunc and C-style astype on values inside the range."""
    x = np.array([0.0, 0.5, 0.999, 1.0, 1.5, 2.5, -0.5, -0.999, -1.0, -1.5, -2.5, 254.9, 255.0, 1e6 + 0.75, -1e6 - 0.75])
    want_i32 = np.array([0, 0, 0, 1, 1, 2, 0, 0, -1, -1, -2, 254, 255, 1000000, -1000000], dtype=np.float64)
    assert np.array_equal(orc.cast_to_int(x, "i32"), want_i32)
    assert np.array_equal(orc.cast_to_int(x, "i32"), np.trunc(x))
    assert np.array_equal(orc.cast_to_int(x, "i32"), x.astype(np.int32).astype(np.float64))
    # u8: the same inside 0..255; outside, the nearest bound
    assert np.array_equal(orc.cast_to_int(np.array([0.2, 7.9, 255.0, 255.9, 300.0, -3.0]), "u8"), np.array([0, 7, 255, 255, 255, 0.0]))
    assert not np.any(np.signbit(orc.cast_to_int(np.array([-0.5, -0.0]), "i32")))    # one zero
    rng = np.random.default_rng(3)
    r = rng.uniform(-1e5, 1e5, 10000)
    assert np.array_equal(orc.cast_to_int(r, "i32"), np.trunc(r))


def test_integer_outputs_of_cast_compare_and_isfinite():
    p = wl.OpProgram("ints")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.cast(p.scalar("muls", a, 10.0), "i32"), "i32")       # (int)(10 a)
    p.output(p.compare("gt", a, b), "u8")                              # a > b as 0 / 1
    p.output(p.unary("isfinite", p.binary("div", a, b)), "u8")
    p.output(p.scalar("muls", a, 10.0), "i32")                         # the store itself casts
    av = np.array([[0.26, -0.26, 1.0, -7.77]]); bv = np.array([[0.25, 0.0, 1.0, 0.0]])
    o = orc.evaluate(p.nodes, [av, bv])
    assert np.array_equal(o[0], [[2, -2, 10, -77]])
    assert np.array_equal(o[1], [[1, 0, 0, 0]])
    assert np.array_equal(o[2], [[1, 0, 1, 0]])                        # -0.26 / 0 and -7.77 / 0 are infinite
    assert np.array_equal(o[3], o[0])
    # a cast in the middle of a program is a rounding point: (int)(2.7) + 0.5 = 2.5
    q = wl.OpProgram("mid")
    x = q.input("f32", 1)
    q.output(q.scalar("adds", q.cast(x, "i32"), 0.5), "f32")
    assert np.array_equal(orc.evaluate(q.nodes, [np.array([2.7, -2.7])])[0], [2.5, -1.5])
