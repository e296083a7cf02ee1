"""Parity at the full sizes of the sweeps, in the launch configuration bench.py times: the largest
instances are too big for the oracle as a whole, but their rows are independent, so contiguous blocks of
rows (the start, the middle around the 2^30-byte offset, the end up to the 2^31-byte boundary, blocks that
straddle a (batch, head) slice) are streamed through the oracle and compared element by element, next to a
random sample of single rows."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc
from tests.parity_util import gate_errors

pytestmark = pytest.mark.gpu


def _sample_rows(n, k, seed, extra=()):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([[0, n - 1], np.asarray(extra, dtype=np.int64), rng.integers(0, n, k)]))


@pytest.mark.parametrize("rows", [262144, 32 * 8192 - 4097])
def test_add_rmsnorm_max_rows_sampled(rows):
    """Config 2 at its largest instance (B = 32, S = 8192: 2 GiB per tensor) and a ragged neighbour."""
    H = 4096
    x = wl.randn((rows, H), torch.bfloat16, 11, "cuda")
    res = wl.randn((rows, H), torch.bfloat16, 12, "cuda")
    w = wl.randn((H,), torch.bfloat16, 13, "cuda", mean=1.0, std=0.02)
    y = torch.full((rows, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    h = torch.full((rows, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    prog = wl.program_add_rmsnorm(H)
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [(rows, H), (rows, H), (H,)])
    dvm.launch(code, [x, res, w, y, h])
    assert dvm.last_device_status() == 0
    idx = _sample_rows(rows, 60, 1, extra=[255, 256, rows // 2])
    ti = torch.from_numpy(idx).cuda()
    want = orc.evaluate(prog.nodes, [wl.to_f64(x[ti]), wl.to_f64(res[ti]), wl.to_f64(w)])
    for got, ref in zip((y, h), want):
        g1, g2 = gate_errors(wl.to_f64(got[ti]), ref)
        assert g2 <= 2e-2, (g1, g2)
    # contiguous blocks of 4096 rows, every element: a tile written to the wrong row cannot hide between samples.
    # Row r starts at byte 8192 r of each tensor: the middle block straddles the 2^30-byte offset, the last block
    # ends at the tensor's end (the 2^31-byte boundary when rows = 262144).
    nb = 4096
    for r0 in (0, (1 << 30) // (2 * H) - nb // 2, rows - nb):
        want = orc.evaluate(prog.nodes, [wl.to_f64(x[r0:r0 + nb]), wl.to_f64(res[r0:r0 + nb]), wl.to_f64(w)])
        for got, ref in zip((y, h), want):
            g1, g2 = gate_errors(wl.to_f64(got[r0:r0 + nb]), ref)
            assert g2 <= 2e-2, (r0, g1, g2)
    # every row was written: no poison left anywhere
    assert not torch.isnan(y.float().sum()) and not torch.isnan(h.float().sum())


@pytest.mark.parametrize("B,S", [(8, 2048), (8, 2047), (3, 1531)])
def test_masked_softmax_max_size_sampled(B, S):
    """Config 3 at its largest instance (B = 8, S = 2048: 2^30 scores) and unaligned neighbours."""
    Hh = 32
    scores = wl.randn((B, Hh, S, S), torch.bfloat16, 21, "cuda")
    mask = wl.causal_mask(S, "cuda")
    out = torch.full((B, Hh, S, S), float("nan"), dtype=torch.bfloat16, device="cuda")
    prog = wl.program_masked_softmax(128)
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [(B, Hh, S, S), (1, 1, S, S)])
    dvm.launch(code, [scores, mask, out])
    assert dvm.last_device_status() == 0
    n_rows = B * Hh * S
    idx = _sample_rows(n_rows, 60, 2, extra=[S - 1, S, n_rows // 2])
    flat_s, flat_o = scores.view(n_rows, S), out.view(n_rows, S)
    ti = torch.from_numpy(idx).cuda()
    sc = wl.to_f64(flat_s[ti])                       # [k, S]
    mk = wl.to_f64(mask.view(S, S)[ti % S])          # the mask row of each sampled query position
    got = wl.to_f64(flat_o[ti])
    for r in range(len(idx)):                        # the oracle, one sampled row at a time
        ref = orc.evaluate(prog.nodes, [sc[r].reshape(1, 1, 1, S), mk[r].reshape(1, 1, 1, S)])[0].reshape(S)
        g1, g2 = gate_errors(got[r], ref)
        assert g2 <= 2e-2, (idx[r], g1, g2)
        q = int(idx[r] % S)
        assert np.all(got[r][q + 1:] == 0)           # masked entries exactly zero
    # contiguous blocks of rows, every element: the first (batch, head) slice, a block across the boundary of
    # two slices in the middle (where the 2^31-byte offset lies when B = 8, S = 2048), the last rows
    nb = min(S, 1024)
    mid = (B * Hh // 2) * S
    for r0 in (0, mid - nb // 2, n_rows - nb):
        rows_i = torch.arange(r0, r0 + nb, device="cuda")
        sc = wl.to_f64(flat_s[r0:r0 + nb]).reshape(nb, 1, 1, S)
        mk = wl.to_f64(mask.view(S, S)[rows_i % S]).reshape(nb, 1, 1, S)
        ref = orc.evaluate(prog.nodes, [sc, mk])[0].reshape(nb, S)
        got = wl.to_f64(flat_o[r0:r0 + nb])
        g1, g2 = gate_errors(got, ref)
        assert g2 <= 2e-2, (r0, g1, g2)
        assert np.array_equal(got == 0, ref == 0)    # masked entries, and only they, are exactly zero
    assert not torch.isnan(out.float().sum())


@pytest.mark.parametrize("B,S", [(16, 7640), (31, 3943)])
def test_head_transpose_view_full_size_sampled(B, S):
    """The views sweep at its largest instances (about 0.5 G elements per tensor): x read through the head
    transpose view; sampled (b, h, s) rows against the oracle's ViewLoad + program, one by one."""
    H, D = 32, 128
    n = B * S * H * D
    xs = wl.randn((n,), torch.bfloat16, 21, "cuda")
    y = wl.randn((n,), torch.bfloat16, 22, "cuda")
    out = torch.full((n,), float("nan"), dtype=torch.bfloat16, device="cuda")
    prog = wl.program_head_transpose_add()
    shp = (B, H, S, D)
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [shp, shp], in_strides=[[S * H * D, D, H * D, 1], None])
    dvm.launch(code, [xs, y, out])
    assert dvm.last_device_status() == 0
    rows = _sample_rows(B * H * S, 200, 3, extra=[S - 1, S, H * S - 1, H * S])
    for r in rows:
        b, h, s_ = int(r // (H * S)), int((r // S) % H), int(r % S)
        src = ((b * S + s_) * H + h) * D
        xrow = orc.view_load(wl.to_f64(xs[src:src + D]), 0, (1, 1, 1, D), (0, 0, 0, 1))
        yrow = wl.to_f64(y[r * D:(r + 1) * D]).reshape(1, 1, 1, D)
        want = orc.evaluate(prog.nodes, [xrow, yrow])[0]
        g1, g2 = gate_errors(wl.to_f64(out[r * D:(r + 1) * D]).reshape(1, D), want.reshape(1, D))
        assert g2 <= 2e-2, (r, g1, g2)
    assert not torch.isnan(out.float().sum())   # every element was written


@pytest.mark.parametrize("shape", [(256, 512, 1024), (251, 509, 1049)])
def test_if_else_add_full_size_sampled(shape):
    """The if-else-add sweep at its size limit (2^27 elements per tensor; the second shape has an odd element
    count): the one-slot launch on three CTAs per SM.  Sampled rows against the oracle one by one; 2x, 4x and
    the add are exact or correctly rounded, so the whole output also equals its fp32 closed form bit for bit."""
    b, s, f = shape
    prog = wl.program_if_else_add()
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [shape] * 4)
    ins = [wl.randn(shape, torch.float32, 70 + i, "cuda") for i in range(4)]
    out = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
    dvm.launch(code, ins + [out])
    assert dvm.last_device_status() == 0
    v = dvm.last_launch_variant()
    assert v["single"] == 1 and v["ctas"] == 3 and v["lean"] == 9   # torch's allocations are 16-byte aligned
    rows = _sample_rows(b * s, 150, 4, extra=[s - 1, s, b * s - 2])
    sub = [t.reshape(-1, f)[torch.as_tensor(rows, device="cuda")].cpu() for t in ins]
    want = orc.evaluate(prog.nodes, [wl.to_f64(x).reshape(1, len(rows), f) for x in sub])[0].reshape(len(rows), f)
    got = wl.to_f64(out.reshape(-1, f)[torch.as_tensor(rows, device="cuda")])
    assert float(np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-30))) <= 1e-6   # (the oracle does not round to fp32)
    ref = torch.where(ins[0] > ins[1], 2 * ins[2], 4 * ins[2])
    ref = (ref.double() + ins[3].double()).float()
    assert torch.equal(out, ref)
