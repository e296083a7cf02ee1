"""Helpers shared by the parity tests: run a program through the C-ABI on the GPU,
evaluate the same inputs with the CPU oracle, and apply the tolerance gates.

Gates (strict elementwise relative error is out of reach of any fp32 evaluation where a program cancels --
exp(ab+c)-a, x-mean, x*w+b -- so the first gate scales by the row maximum):
  G1  |g - o| <= R * max(|o|, max_j |o_row_j|)   every program, every element
  G2  |g - o| <= R * |o|                          programs without subtractive cancellation
  G3  exact                                       structural zeros / integer outputs
with R = 1e-5 for fp32 programs and 2e-2 for bf16 programs.  Non-finite oracle
values must be matched in class and sign.
"""
from __future__ import annotations

import numpy as np
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16, "u8": torch.uint8, "i32": torch.int32}
R_TOL = {"f32": 1e-5, "bf16": 2e-2}


def program_dtype(prog: wl.OpProgram) -> str:
    """bf16 if any tensor of the program is bf16 (the looser tolerance applies), else f32."""
    kinds = [n[1] for n in prog.nodes if n[0] == "input"] + [n[2] for n in prog.nodes if n[0] == "output"]
    return "bf16" if "bf16" in kinds else "f32"


def gpu_run(prog: wl.OpProgram, inputs, params=(), stream=None, poison=True):
    """Encode for the inputs' shapes, launch once, return (outputs, code)."""
    p = dvm.program_from_nodes(prog.nodes)
    dev_in = [t.cuda() for t in inputs]
    code = dvm.encode(p, [tuple(t.shape) for t in dev_in], params)
    outs = []
    for shp, node in zip(code.out_shapes, prog.output_nodes):
        o = torch.empty(shp, dtype=TORCH_DT[node[2]], device="cuda")
        if poison:
            o.fill_(float("nan") if o.dtype.is_floating_point else 123)
        outs.append(o)
    torch.cuda.synchronize()
    dvm.launch(code, dev_in + outs, stream)
    assert dvm.last_device_status(stream) == 0
    return outs, code


def oracle_run(prog: wl.OpProgram, inputs, params=()):
    return orc.evaluate(prog.nodes, [wl.to_f64(t) for t in inputs], params)


def gate_errors(got: np.ndarray, want: np.ndarray):
    """Returns (g1_err, g2_err): max over elements of |g-o| / scale for both denominators."""
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    fin = np.isfinite(want)
    # non-finite values: same class and sign
    assert np.array_equal(np.isnan(got), np.isnan(want)), "NaN pattern differs"
    inf = np.isinf(want)
    assert np.array_equal(got[inf], want[inf]), "infinities differ"
    if want.size == 0:
        return 0.0, 0.0
    diff = np.where(fin, np.abs(got - np.where(fin, want, 0.0)), 0.0)
    absw = np.where(fin, np.abs(want), 0.0)
    rowmax = np.max(absw, axis=-1, keepdims=True) if want.ndim else absw
    den1 = np.maximum(absw, rowmax)
    with np.errstate(divide="ignore", invalid="ignore"):
        g1 = np.where(diff == 0, 0.0, diff / den1)
        g2 = np.where(diff == 0, 0.0, diff / absw)
    return float(np.max(g1)), float(np.max(g2))


# Statistics reported beside the gates for the programs whose strict elementwise error no fp32 evaluation can
# bound (C1, C4 GELU, C4 LayerNorm, C5): filled by the tests, printed in pytest's terminal summary.
STRICT_REPORT = []


def strict_stats(got, want, want_fp32, r):
    """Strict elementwise relative error of `got` against the float64 oracle `want`: its maximum, how many
    elements exceed r, and how many of those lie among the elements a faithful fp32 evaluation already gets
    right (|o32 - o64| <= 1e-6 |o64|: "well conditioned").  Reported, not gated: the row-scaled gate cannot see
    a small output that was zeroed, this count can."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    w32 = np.asarray(want_fp32, dtype=np.float64).reshape(-1)
    fin = np.isfinite(want) & (want != 0)
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(fin, np.abs(got - want) / np.abs(want), 0.0)
        well = fin & (np.abs(w32 - want) <= 1e-6 * np.abs(want))
    over = rel > r
    return {"n": int(want.size), "strict_max": float(rel.max()) if want.size else 0.0, "n_over": int(over.sum()),
            "n_well": int(well.sum()), "n_over_well": int((over & well).sum()),
            "well_max": float(rel[well].max()) if well.any() else 0.0}


def record_strict(label, prog, got_list, inputs, params=(), want_list=None):
    """Computes strict_stats for every output of a program run and appends them to STRICT_REPORT."""
    r = R_TOL[program_dtype(prog)]
    ins64 = [wl.to_f64(t) for t in inputs]
    if want_list is None:
        want_list = orc.evaluate(prog.nodes, ins64, params)
    want32 = orc.evaluate(prog.nodes, ins64, params, diagnostic_fp32=True)
    out = []
    for g, w, w32 in zip(got_list, want_list, want32):
        st = strict_stats(wl.to_f64(g) if isinstance(g, torch.Tensor) else g, w, w32, r)
        st["label"] = label
        st["r"] = r
        STRICT_REPORT.append(st)
        out.append(st)
    return out


def check(prog, got_list, want_list, strict=False, tol=None):
    r = tol if tol is not None else R_TOL[program_dtype(prog)]
    worst = (0.0, 0.0)
    for g, w in zip(got_list, want_list):
        g1, g2 = gate_errors(wl.to_f64(g) if isinstance(g, torch.Tensor) else g, w)
        assert g1 <= r, f"{prog.name}: G1 error {g1:.3e} > {r:.1e}"
        if strict:
            assert g2 <= r, f"{prog.name}: G2 (strict) error {g2:.3e} > {r:.1e}"
        worst = (max(worst[0], g1), max(worst[1], g2))
    return worst
