"""CPU oracle for the DVM hot path -- TEST INFRASTRUCTURE, not a product path.

What the device-side virtual machine must produce is, by construction of the
method, the same tensors as evaluating the fused program's basic operators one
after another on whole tensors: fusion only replaces global-memory round trips
by local memory (Sec. 5.1, "Pattern-based fusion") and tiling only partitions
the iteration space (Sec. 4.2, "Shape tiling").  So this oracle is that plain
definition: it walks the op program in order and materialises every
intermediate as a whole float64 numpy array.  No tiling, no fusion, no
bytecode, no blocking.  It shares no code with the encoder or the CUDA
kernels and imports nothing from the product package.

Arithmetic: every value is float64.  bf16 / fp32 inputs are widened exactly by
the caller.  A "cast" node in the middle of a program is a semantic rounding
point (Table 1, Cast) and rounds to the target format (nearest-even) before
widening again; the device's implicit fp32 working precision is NOT emulated.
Outputs are returned unrounded in float64.

Per-node definitions follow Table 1 ("Tile-level Virtual Instructions"):
  Add/Sub/Mul/Div/Min/Max  elementwise                       (Table 1, binary rows)
  Adds/Muls                x op scalar                        (Table 1, Adds/Muls)
  Sqrt/Abs/Log/Exp/Round/Floor                                (Table 1, unary rows)
  Cast                     (dst_dtype)(x); to an integer type   (Table 1, Cast)
                           the fraction is dropped (toward zero)
  Sum/Max/Min reduce       [M,size,N] -> [M,1,N]; N = 1 unless a  (Table 1, Sum/Max/Min)
                           reduce node names another axis
  Broadcast                implicit in numpy-style broadcasting (Table 1, Broadcast)
  Cmp                      1.0 where the relation holds, else 0.0  (Table 1, Cmp)
  Select                   cond != 0 ? x : y                       (Table 1, Select)
  ViewLoad / ViewStore     element (i_0..i_{d-1}) of a view lies at          (Table 1, ViewLoad / ViewStore:
                           base + sum_k i_k * stride_k of its storage        non-contiguous tiles, per-dim strides)
                           (view_load / view_store below; evaluate() itself sees logical arrays only)
Extensions that the benchmark programs need and Table 1 lacks: erf, sigmoid(x) = 1/(1+exp(-x)), rsqrt(x) = 1/sqrt(x),
recip, neg, tanh, and matmul C[i,j] = sum_k A[i,k] B[k,j] (the paper's cube
operation, Sec. 4.2, described in prose only).

Pins (tests/test_oracle_pins.py): closed forms (softmax rows sum to 1, causal
row i is 1/(i+1) for equal scores, RMSNorm unit RMS, LayerNorm zero mean /
unit variance, GELU/sigmoid identities), torch float64 library routines on the
special cases they cover, a pure-Python scalar evaluator on tiny inputs, and a
triple-loop matmul.  NaN propagation in min/max, pow and log of non-positive
numbers are "parity unpinned".
"""
from __future__ import annotations

import numpy as np
from scipy import special as _special

__all__ = ["evaluate", "round_to_bf16", "round_to_f32", "cast_to_int"]


def round_to_f32(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 to the fp32 grid, returned as float64."""
    with np.errstate(over="ignore"):
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 to the bfloat16 grid, returned as float64.

    bf16 is the top 16 bits of an fp32 word.  Rounding goes through fp32; when
    the fp32 value sits exactly on a bf16 tie although x did not, the tie is
    broken towards x so that the result is the single correct rounding of x.
    """
    x = np.asarray(x, dtype=np.float64)
    with np.errstate(over="ignore"):
        y = x.astype(np.float32)
    u = y.view(np.uint32).astype(np.uint64)
    low = u & 0xFFFF
    base = u & 0xFFFF0000
    up = base + 0x10000
    is_tie = low == 0x8000
    # direction of the discarded part of x relative to the fp32 value y
    mag_gt = np.abs(x) > np.abs(y.astype(np.float64))
    mag_lt = np.abs(x) < np.abs(y.astype(np.float64))
    even_up = ((u >> 16) & 1) == 1
    round_up = np.where(is_tie, np.where(mag_gt, True, np.where(mag_lt, False, even_up)),
                        low > 0x8000)
    r = np.where(round_up, up, base).astype(np.uint32)
    out = r.view(np.float32).astype(np.float64)
    # NaN / inf keep their class
    out = np.where(np.isnan(x), np.nan, out)
    out = np.where(np.isinf(x), x, out)
    return out.reshape(x.shape)


_INT_RANGE = {"i32": (-2147483648.0, 2147483647.0), "u8": (0.0, 255.0)}


def cast_to_int(x: np.ndarray, dtype: str) -> np.ndarray:
    """Table 1, Cast to an integer type: the fraction is dropped (rounding toward zero, the conversion C defines);
    the result is returned as float64 holding the integer.  Values outside the type's range take the nearest
    bound and NaN becomes 0 -- the paper fixes neither ("parity unpinned"; the sweeps stay inside the range)."""
    lo, hi = _INT_RANGE[dtype]
    x = np.asarray(x, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        t = np.where(x < 0, np.ceil(x), np.floor(x))          # toward zero, written out
        t = np.where(np.isnan(x), 0.0, np.minimum(np.maximum(t, lo), hi))
    return t + 0.0                                            # (-0 -> +0: an integer has one zero)


def _round_to(x, dtype):
    if dtype == "f32":
        return round_to_f32(x)
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype in _INT_RANGE:
        return cast_to_int(x, dtype)
    raise ValueError(f"unknown dtype {dtype}")


_UNARY = {
    "exp": np.exp,                                   # Table 1, Exp
    "sqrt": np.sqrt,                                 # Table 1, Sqrt
    "abs": np.abs,                                   # Table 1, Abs
    "log": np.log,                                   # Table 1, Log
    "floor": np.floor,                               # Table 1, Floor
    "round": np.rint,                                # Table 1, Round (half to even)
    "rsqrt": lambda x: 1.0 / np.sqrt(x),             # extension
    "erf": _special.erf,                             # extension
    "sigmoid": lambda x: 1.0 / (1.0 + np.exp(-x)),   # extension
    "neg": lambda x: -x,                             # extension
    "recip": lambda x: 1.0 / x,                      # extension
    "tanh": np.tanh,                                 # extension
    "isfinite": lambda x: np.isfinite(x).astype(np.float64),   # Table 1, IsFinite: 1 for a finite value, else 0
}

_BINARY = {
    "add": lambda a, b: a + b,                       # Table 1, Add
    "sub": lambda a, b: a - b,                       # Table 1, Sub
    "mul": lambda a, b: a * b,                       # Table 1, Mul
    "div": lambda a, b: a / b,                       # Table 1, Div
    "max": lambda a, b: np.where(a > b, a, b),       # Table 1, Max
    "min": lambda a, b: np.where(a < b, a, b),       # Table 1, Min
    "pow": lambda a, b: np.power(a, b),              # Table 1, Pow: a ** b (IEEE pow: NaN for a negative base
                                                     # with a non-integer exponent)
}

_COMPARE = {                                         # Table 1, Cmp: 1 where the relation holds, else 0
    "gt": lambda a, b: (a > b).astype(np.float64),
    "ge": lambda a, b: (a >= b).astype(np.float64),
    "lt": lambda a, b: (a < b).astype(np.float64),
    "le": lambda a, b: (a <= b).astype(np.float64),
    "eq": lambda a, b: (a == b).astype(np.float64),
    "ne": lambda a, b: (a != b).astype(np.float64),
}

_REDUCE = {
    # Table 1, Sum / Max / Min: [M, size, N] -> [M, 1, N]; the reduced dim is `axis`, counted from the end
    # (-1: the last dim, N = 1; -2: the paper's penultimate dim), and stays with size 1
    "sum": lambda x, axis=-1: np.sum(x, axis=axis, keepdims=True),
    "max": lambda x, axis=-1: np.max(x, axis=axis, keepdims=True),
    "min": lambda x, axis=-1: np.min(x, axis=axis, keepdims=True),
}


def evaluate(nodes, inputs, params=(), diagnostic_fp32=False):
    """Evaluate an op program node by node on whole tensors.

    nodes  : list of node tuples (see the workload module's docstring).
    inputs : float64 numpy arrays, one per "input" node, in order; shapes may
             broadcast against each other numpy-style (right-aligned).
    params : runtime scalar arguments referenced by ("param", k).
    Returns the list of outputs (float64, unrounded), in "output"-node order.

    diagnostic_fp32=True runs the same steps with every value held in float32
    instead of float64.  That is NOT the reference: it only labels the elements
    on which a faithful fp32 evaluation already agrees with the float64 result
    ("well conditioned"), for the statistics the parity tests report beside
    their gates.
    """
    if diagnostic_fp32:
        outs32 = _evaluate(nodes, inputs, params, np.float32)
        return [o.astype(np.float64) for o in outs32]
    return _evaluate(nodes, inputs, params, np.float64)


def _evaluate(nodes, inputs, params, ft):
    vals = [None] * len(nodes)
    outs = []
    it = iter(inputs)
    with np.errstate(all="ignore"):
        for i, n in enumerate(nodes):
            kind = n[0]
            if kind == "input":
                a = np.asarray(next(it), dtype=ft)
                if a.ndim != n[2]:
                    raise ValueError(f"input node {i}: rank {a.ndim} != declared {n[2]}")
                vals[i] = a
            elif kind == "unary":
                vals[i] = _UNARY[n[1]](vals[n[2]])
            elif kind == "binary":
                vals[i] = _BINARY[n[1]](vals[n[2]], vals[n[3]])
            elif kind == "scalar":
                s = n[3]
                # the scalar is an fp32 immediate widened exactly (Table 1, Adds/Muls)
                s = ft(np.float32(params[s[1]] if isinstance(s, tuple) else s))
                vals[i] = vals[n[2]] + s if n[1] == "adds" else vals[n[2]] * s
            elif kind == "cast":
                vals[i] = _round_to(vals[n[1]], n[2]).astype(ft)
            elif kind == "reduce":
                axis = n[3] if len(n) > 3 else -1
                if not (-vals[n[2]].ndim <= axis <= -1):
                    raise ValueError("reduce axis counts from the end: -1 .. -rank")
                vals[i] = _REDUCE[n[1]](vals[n[2]], axis)
            elif kind == "matmul":
                vals[i] = np.matmul(vals[n[1]], vals[n[2]])
            elif kind == "compare":
                vals[i] = _COMPARE[n[1]](*np.broadcast_arrays(vals[n[2]], vals[n[3]])).astype(ft)
            elif kind == "select":                   # Table 1, Select: cond ? x : y, cond = (value != 0)
                c, x, y = np.broadcast_arrays(vals[n[1]], vals[n[2]], vals[n[3]])
                vals[i] = np.where(c != 0, x, y)
            elif kind == "output":
                # an output stored as an integer type holds the integer the cast gives (Table 1, Cast; Cmp and
                # IsFinite values are 0 / 1 already); floating outputs are returned unrounded
                v = vals[n[1]]
                outs.append(np.array(cast_to_int(v, n[2]) if n[2] in _INT_RANGE else v, dtype=ft))
            else:
                raise ValueError(f"unknown node kind {kind}")
    return outs


def _view_index(offset, shape, strides):
    """Flat storage index of every element of a view: offset + sum_k i_k * stride_k (Table 1, ViewLoad)."""
    shape = tuple(int(d) for d in shape)
    strides = tuple(int(t) for t in strides)
    if len(shape) != len(strides):
        raise ValueError("one stride per dim")
    idx = np.full(shape, int(offset), dtype=np.int64)
    for k, (d, t) in enumerate(zip(shape, strides)):
        ik = np.arange(d, dtype=np.int64).reshape([d if j == k else 1 for j in range(len(shape))])
        idx = idx + ik * t
    return idx


def view_load(storage: np.ndarray, offset: int, shape, strides) -> np.ndarray:
    """ViewLoad (Table 1): the logical array a strided view denotes.  `storage` is the flat buffer, `offset`
    and `strides` are in elements; a stride of 0 repeats the element (broadcast)."""
    flat = np.asarray(storage).reshape(-1)
    idx = _view_index(offset, shape, strides)
    if idx.size and (idx.min() < 0 or idx.max() >= flat.size):
        raise IndexError("view reaches outside its storage")
    return flat[idx]


def view_store(storage: np.ndarray, offset: int, shape, strides, values: np.ndarray) -> np.ndarray:
    """ViewStore (Table 1): a copy of `storage` with the view's elements replaced by `values`; every other
    element keeps its value.  The view must not alias itself (two index tuples, one address)."""
    flat = np.array(storage, copy=True).reshape(-1)
    idx = _view_index(offset, shape, strides)
    if idx.size and (idx.min() < 0 or idx.max() >= flat.size):
        raise IndexError("view reaches outside its storage")
    if np.unique(idx).size != idx.size:
        raise ValueError("a stored view must address every element once")
    flat[idx.reshape(-1)] = np.asarray(values).reshape(-1)
    return flat.reshape(np.asarray(storage).shape)
