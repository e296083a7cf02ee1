"""Seeded synthetic inputs for the DVM hot path: op programs (as plain data),
dynamic-shape samplers and tensor generators.

This module is the one piece shared by the CUDA path's tests/bench and by the
CPU oracle's tests.  It holds *inputs only*: an op program here is a list of
tuples naming basic operators (the "computation graph of basic operators to
fuse" that the paper's bytecode compiler receives, Sec. 3 "Operator
Compiler"), shapes are integers drawn from a seeded generator, tensors are
seeded random draws.  None of the method's arithmetic (no evaluation, no
tiling, no encoding) lives here.

Program node tuples (value ids are positions in ``nodes``):
    ("input",  dtype, rank)
    ("unary",  op, x)                 op in UNARY_OPS
    ("binary", op, x, y)              op in BINARY_OPS, numpy-style broadcasting
    ("scalar", op, x, s)              op in SCALAR_OPS; s is a float immediate or
                                      ("param", k): k-th runtime scalar argument
    ("cast",   x, dtype)
    ("reduce", op, x[, axis])         op in REDUCE_OPS, keepdim; axis counts from the end (default -1: the last
                                      axis; -2: the penultimate one, Table 1's [M,size,N] -> [M,1,N])
    ("matmul", a, b)                  [M,K] x [K,N]
    ("output", x, dtype)              marks value x as an output stored as dtype

The workloads follow the five benchmark configurations: their shape ranges are
those of the paper's LLM-derived workloads (Table 2: hidden 4096, FFN 11008,
sequence up to 8192), the values are plain Gaussian / uniform draws standing
in for real activations and weights.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np
import torch

UNARY_OPS = ("exp", "sqrt", "rsqrt", "abs", "log", "erf", "sigmoid", "neg",
             "recip", "floor", "round", "tanh", "isfinite")
BINARY_OPS = ("add", "sub", "mul", "div", "min", "max", "pow")
SCALAR_OPS = ("adds", "muls")
REDUCE_OPS = ("sum", "max", "min")
COMPARE_OPS = ("gt", "ge", "lt", "le", "eq", "ne")
DTYPES = ("f32", "bf16")
INT_DTYPES = ("u8", "i32")   # outputs and casts only (Table 1: Cast; Cmp / IsFinite results stored as 0 / 1)


@dataclass
class OpProgram:
    """A shape-agnostic fused operator program, as plain data."""
    name: str = "program"
    nodes: List[tuple] = field(default_factory=list)
    n_params: int = 0

    def _push(self, node) -> int:
        self.nodes.append(tuple(node))
        return len(self.nodes) - 1

    def input(self, dtype: str, rank: int) -> int:
        assert dtype in DTYPES
        return self._push(("input", dtype, rank))

    def unary(self, op: str, x: int) -> int:
        assert op in UNARY_OPS
        return self._push(("unary", op, x))

    def binary(self, op: str, x: int, y: int) -> int:
        assert op in BINARY_OPS
        return self._push(("binary", op, x, y))

    def scalar(self, op: str, x: int, s) -> int:
        assert op in SCALAR_OPS
        if isinstance(s, tuple):
            assert s[0] == "param"
            self.n_params = max(self.n_params, s[1] + 1)
        return self._push(("scalar", op, x, s))

    def cast(self, x: int, dtype: str) -> int:
        assert dtype in DTYPES + INT_DTYPES
        return self._push(("cast", x, dtype))

    def reduce(self, op: str, x: int, axis: int = -1) -> int:
        assert op in REDUCE_OPS and axis <= -1
        return self._push(("reduce", op, x) if axis == -1 else ("reduce", op, x, axis))

    def matmul(self, a: int, b: int) -> int:
        return self._push(("matmul", a, b))

    def compare(self, op: str, x: int, y: int) -> int:
        assert op in COMPARE_OPS
        return self._push(("compare", op, x, y))

    def select(self, cond: int, x: int, y: int) -> int:
        return self._push(("select", cond, x, y))

    def output(self, x: int, dtype: str) -> int:
        assert dtype in DTYPES + INT_DTYPES
        return self._push(("output", x, dtype))

    @property
    def input_ids(self) -> List[int]:
        return [i for i, n in enumerate(self.nodes) if n[0] == "input"]

    @property
    def output_nodes(self) -> List[tuple]:
        return [n for n in self.nodes if n[0] == "output"]


# --------------------------------------------------------------------------
# The op programs of the five configurations (definitions: standard ones;
# where a configuration is silent the reading taken is stated in the program's
# docstring: norm on the un-rounded fp32 sum, exact-erf GELU, LayerNorm without
# affine parameters and with biased variance, mask added before the scale).
# --------------------------------------------------------------------------

def program_c1() -> OpProgram:
    """out = exp(a*b + c) - a, fp32."""
    p = OpProgram("c1_elementwise")
    a, b, c = p.input("f32", 2), p.input("f32", 2), p.input("f32", 2)
    t = p.binary("mul", a, b)
    t = p.binary("add", t, c)
    t = p.unary("exp", t)
    t = p.binary("sub", t, a)
    p.output(t, "f32")
    return p


def program_add_rmsnorm(hidden: int = 4096, eps: float = 1e-6) -> OpProgram:
    """h = x + res; y = h * rsqrt(mean(h*h) + eps) * w.  Outputs (y, h), bf16."""
    p = OpProgram("add_rmsnorm")
    x, res, w = p.input("bf16", 2), p.input("bf16", 2), p.input("bf16", 1)
    h = p.binary("add", x, res)
    sq = p.binary("mul", h, h)
    ms = p.reduce("sum", sq)
    ms = p.scalar("muls", ms, 1.0 / hidden)
    ms = p.scalar("adds", ms, eps)
    r = p.unary("rsqrt", ms)
    y = p.binary("mul", h, r)
    y = p.binary("mul", y, w)
    p.output(y, "bf16")
    p.output(h, "bf16")
    return p


def program_masked_softmax(head_dim: int = 128) -> OpProgram:
    """softmax((scores + mask) / sqrt(head_dim)) over the last axis, bf16 in/out."""
    p = OpProgram("masked_softmax")
    s, m = p.input("bf16", 4), p.input("bf16", 4)
    z = p.binary("add", s, m)
    z = p.scalar("muls", z, 1.0 / math.sqrt(head_dim))
    mx = p.reduce("max", z)
    e = p.unary("exp", p.binary("sub", z, mx))
    den = p.reduce("sum", e)
    p.output(p.binary("div", e, den), "bf16")
    return p


def program_gelu_affine() -> OpProgram:
    """t = x*w + b; out = 0.5*t*(1 + erf(t/sqrt(2))), fp32; w, b are [1, cols]."""
    p = OpProgram("gelu_affine")
    x, w, b = p.input("f32", 2), p.input("f32", 2), p.input("f32", 2)
    t = p.binary("add", p.binary("mul", x, w), b)
    u = p.unary("erf", p.scalar("muls", t, 1.0 / math.sqrt(2.0)))
    u = p.scalar("adds", u, 1.0)
    o = p.scalar("muls", p.binary("mul", t, u), 0.5)
    p.output(o, "f32")
    return p


def program_layernorm(eps: float = 1e-5) -> OpProgram:
    """LayerNorm over the last axis, no affine, biased variance, two-pass.
    Runtime scalar argument 0 is 1/cols."""
    p = OpProgram("layernorm")
    x = p.input("f32", 2)
    mu = p.scalar("muls", p.reduce("sum", x), ("param", 0))
    d = p.binary("sub", x, mu)
    v = p.scalar("muls", p.reduce("sum", p.binary("mul", d, d)), ("param", 0))
    r = p.unary("rsqrt", p.scalar("adds", v, eps))
    p.output(p.binary("mul", d, r), "f32")
    return p


def program_sigmoid_mul() -> OpProgram:
    """out = sigmoid(x) * y, fp32."""
    p = OpProgram("sigmoid_mul")
    x, y = p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("mul", p.unary("sigmoid", x), y), "f32")
    return p


def program_mlp_gate() -> OpProgram:
    """out = SiLU(X @ Wg) * (X @ Wu), bf16 in, fp32 accumulate, bf16 out."""
    p = OpProgram("mlp_gate")
    x, wg, wu = p.input("bf16", 2), p.input("bf16", 2), p.input("bf16", 2)
    g = p.matmul(x, wg)
    u = p.matmul(x, wu)
    o = p.binary("mul", p.binary("mul", g, p.unary("sigmoid", g)), u)
    p.output(o, "bf16")
    return p


def program_if_else_add() -> OpProgram:
    """out = (a > b ? 2x : 4x) + y, fp32: the paper's compound operator with a data-dependent branch
    (Sec. 6, subgraph-level analysis), as Cmp + Select (Table 1)."""
    p = OpProgram("if_else_add")
    a, b, x, y = (p.input("f32", 3) for _ in range(4))
    c = p.compare("gt", a, b)
    s = p.select(c, p.scalar("muls", x, 2.0), p.scalar("muls", x, 4.0))
    p.output(p.binary("add", s, y), "f32")
    return p


def program_if_else_add_mask() -> OpProgram:
    """The same, with the comparison's 0 / 1 also stored, as u8 (Table 1, Cmp: integer output, bit-exact)."""
    p = OpProgram("if_else_add_mask")
    a, b, x, y = (p.input("f32", 3) for _ in range(4))
    c = p.compare("gt", a, b)
    s = p.select(c, p.scalar("muls", x, 2.0), p.scalar("muls", x, 4.0))
    p.output(p.binary("add", s, y), "f32")
    p.output(c, "u8")
    return p


def program_quantise(in_dtype: str = "f32", scale: float = 10.0) -> OpProgram:
    """Table 1, Cast: (int)(scale * x) stored as i32, the same clipped into a byte stored as u8, and the cast value
    used again in fp32 arithmetic ((int)(scale * x) * 0.5)."""
    p = OpProgram("quantise_" + in_dtype)
    x = p.input(in_dtype, 2)
    q = p.cast(p.scalar("muls", x, scale), "i32")
    p.output(q, "i32")
    p.output(p.scalar("adds", p.scalar("muls", x, scale), 128.0), "u8")
    p.output(p.scalar("muls", q, 0.5), "f32")
    return p


def program_head_transpose_add() -> OpProgram:
    """out[b,h,s,:] = 0.5 * x[b,h,s,:] + y[b,h,s,:], bf16 rank 4: the elementwise consumer of an attention head
    transpose.  x is given as a VIEW (stored [B,S,H,D], read as [B,H,S,D]: Table 1, ViewLoad); y, out dense."""
    p = OpProgram("head_transpose_add")
    x, y = p.input("bf16", 4), p.input("bf16", 4)
    p.output(p.binary("add", p.scalar("muls", x, 0.5), y), "bf16")
    return p


def shapes_views(n: int = 60, H: int = 32, D: int = 128, max_tokens: int = 1 << 17) -> List[Tuple[int, int]]:
    """(B, S) per instance: B ~ U{1..32}, S ~ U{1..8192}, redrawn while B*S exceeds max_tokens (the tensors are
    [B,32,S,128] bf16: 8 KB per token)."""
    rng = np.random.default_rng(CFG_SEED["views"])
    out = []
    while len(out) < n:
        b, s_ = int(rng.integers(1, 32, endpoint=True)), int(rng.integers(1, 8192, endpoint=True))
        if b * s_ <= max_tokens:
            out.append((b, s_))
    return out


def program_matmul() -> OpProgram:
    """out = A @ B, bf16 in, fp32 accumulate, bf16 out (Table 2, matmul)."""
    p = OpProgram("matmul")
    a, b = p.input("bf16", 2), p.input("bf16", 2)
    p.output(p.matmul(a, b), "bf16")
    return p


def program_addmm() -> OpProgram:
    """out = A @ B + C with C [m,n]: the paper decomposes addmm into matmul and add (Sec. 3); the add is the
    fused epilogue (cube-vector fusion, Sec. 5.1).  bf16 in, fp32 accumulate, bf16 out."""
    p = OpProgram("addmm")
    a, b, c = p.input("bf16", 2), p.input("bf16", 2), p.input("bf16", 2)
    p.output(p.binary("add", p.matmul(a, b), c), "bf16")
    return p


def program_add_sqrt() -> OpProgram:
    """c = sqrt(a + b): the paper's vector-vector fusion example (Sec. 5.1)."""
    p = OpProgram("add_sqrt")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.unary("sqrt", p.binary("add", a, b)), "f32")
    return p


STACK_KINDS = ("gelu_affine", "layernorm", "sigmoid_mul")


def stack_program(kind: str) -> OpProgram:
    return {"gelu_affine": program_gelu_affine,
            "layernorm": program_layernorm,
            "sigmoid_mul": program_sigmoid_mul}[kind]()


# --------------------------------------------------------------------------
# Seeds, shape samplers
# --------------------------------------------------------------------------
CFG_SEED = {"c1": 0, "c2": 1, "c3": 2, "c4": 3, "c5": 4, "addmm": 5, "ifelse": 6, "views": 7}

# (n, k) pairs "extracted from common LLMs" of the paper's matmul / addmm experiments (Table 2)
LLM_NK = ((4096, 4096), (11008, 4096), (4096, 11008), (5120, 5120), (13696, 5120), (5120, 13696),
          (8192, 8192), (28672, 8192), (8192, 28672))


def _ints(rng, lo, hi, n):
    return [int(v) for v in rng.integers(lo, hi, size=n, endpoint=True)]


def shapes_c2(n: int = 200) -> List[Tuple[int, int]]:
    """(B, S) pairs; rows T = B*S of width 4096."""
    rng = np.random.default_rng(CFG_SEED["c2"])
    return list(zip(_ints(rng, 1, 32, n), _ints(rng, 1, 8192, n)))


def shapes_c3(n: int = 100) -> List[Tuple[int, int]]:
    """(B, S) pairs; scores [B, 32, S, S]."""
    rng = np.random.default_rng(CFG_SEED["c3"])
    return list(zip(_ints(rng, 1, 8, n), _ints(rng, 17, 2048, n)))


def shapes_c4(n_launches: int = 50, n_programs: int = 64):
    """Per launch: list of (kind, rows, cols)."""
    rng = np.random.default_rng(CFG_SEED["c4"])
    out = []
    for _ in range(n_launches):
        kinds = _ints(rng, 0, len(STACK_KINDS) - 1, n_programs)
        rows = _ints(rng, 1, 512, n_programs)
        cols = _ints(rng, 64, 4096, n_programs)
        out.append([(STACK_KINDS[k], r, c) for k, r, c in zip(kinds, rows, cols)])
    return out


def shapes_c5(n: int = 64) -> List[int]:
    rng = np.random.default_rng(CFG_SEED["c5"])
    return _ints(rng, 1, 4096, n)


def shapes_if_else_add(n: int = 50, max_elems: int = 1 << 27) -> List[Tuple[int, int, int]]:
    """(b, s, f) per instance: b ~ U{1..256}, s ~ U{1..512}, f ~ U{1..8192} (Table 2), redrawn while the
    instance exceeds max_elems elements (five fp32 tensors of it must fit the device pools)."""
    rng = np.random.default_rng(CFG_SEED["ifelse"])
    out = []
    while len(out) < n:
        b, s_, f = int(rng.integers(1, 256, endpoint=True)), int(rng.integers(1, 512, endpoint=True)), int(rng.integers(1, 8192, endpoint=True))
        if b * s_ * f <= max_elems:
            out.append((b, s_, f))
    return out


def shapes_addmm(n: int = 36) -> List[Tuple[int, int, int]]:
    """(m, n, k) per instance: m ~ U{1..8192}, (n, k) cycling through the nine pairs of Table 2."""
    rng = np.random.default_rng(CFG_SEED["addmm"])
    ms = _ints(rng, 1, 8192, n)
    return [(m,) + LLM_NK[i % len(LLM_NK)] for i, m in enumerate(ms)]


# --------------------------------------------------------------------------
# Tensor generators (seeded; device may be "cpu" or "cuda")
# --------------------------------------------------------------------------

def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def data_seed(cfg: str, instance: int) -> int:
    return CFG_SEED[cfg] * 1_000_003 + instance


def randn(shape, dtype, seed, device="cpu", mean=0.0, std=1.0) -> torch.Tensor:
    g = _gen(seed, device)
    t = torch.empty(shape, dtype=torch.float32, device=device).normal_(mean, std, generator=g)
    return t.to(dtype)


def uniform(shape, dtype, seed, device="cpu", lo=-1.0, hi=1.0) -> torch.Tensor:
    g = _gen(seed, device)
    t = torch.empty(shape, dtype=torch.float32, device=device).uniform_(lo, hi, generator=g)
    return t.to(dtype)


def inputs_c1(device="cpu"):
    """a, b, c ~ U(-1, 1), fp32 [7, 1531], one generator seeded 0."""
    g = _gen(0, device)
    return [torch.empty((7, 1531), dtype=torch.float32, device=device).uniform_(-1, 1, generator=g)
            for _ in range(3)]


def inputs_add_rmsnorm(rows: int, hidden: int, seed: int, device="cpu"):
    x = randn((rows, hidden), torch.bfloat16, seed, device)
    res = randn((rows, hidden), torch.bfloat16, seed + 7919, device)
    w = randn((hidden,), torch.bfloat16, seed + 104729, device, mean=1.0, std=0.02)
    return [x, res, w]


def causal_mask(S: int, device="cpu") -> torch.Tensor:
    """Additive causal mask [1, 1, S, S]: 0 where j <= i, -inf where j > i."""
    m = torch.zeros((S, S), dtype=torch.float32, device=device)
    m.masked_fill_(torch.ones((S, S), dtype=torch.bool, device=device).triu_(1), float("-inf"))
    return m.to(torch.bfloat16).reshape(1, 1, S, S)


def inputs_masked_softmax(B: int, H: int, S: int, seed: int, device="cpu"):
    return [randn((B, H, S, S), torch.bfloat16, seed, device), causal_mask(S, device)]


def inputs_stack(kind: str, rows: int, cols: int, seed: int, device="cpu"):
    """Returns (tensors, scalar_params) for one stacked program."""
    f32 = torch.float32
    if kind == "gelu_affine":
        return [randn((rows, cols), f32, seed, device),
                randn((1, cols), f32, seed + 1, device),
                randn((1, cols), f32, seed + 2, device)], []
    if kind == "layernorm":
        return [randn((rows, cols), f32, seed, device)], [1.0 / cols]
    if kind == "sigmoid_mul":
        return [randn((rows, cols), f32, seed, device),
                randn((rows, cols), f32, seed + 1, device)], []
    raise ValueError(kind)


def inputs_mlp_gate(M: int, K: int, N: int, seed: int, device="cpu", weights=None):
    x = randn((M, K), torch.bfloat16, seed, device)
    if weights is None:
        weights = mlp_weights(K, N, device)
    return [x, weights[0], weights[1]]


def mlp_weights(K: int, N: int, device="cpu"):
    base = CFG_SEED["c5"] * 1_000_003
    return (randn((K, N), torch.bfloat16, base + 500_001, device, std=0.02),
            randn((K, N), torch.bfloat16, base + 500_002, device, std=0.02))


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a bf16/fp32 tensor to a float64 numpy array (host)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
