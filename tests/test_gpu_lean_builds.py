"""The lean interpreter's specialised builds (one program per launch): which build a launch runs on follows from the
program and its tensors, and every build gives the oracle's result -- the same program on inputs that move it from
one build to the next (a misaligned tensor, a row length that leaves slots empty, a broadcast outer dim)."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


def _run(prog, ins, outs_like=None):
    outs, code = gpu_run(prog, ins)
    want = oracle_run(prog, [t.cpu() for t in ins])
    check(prog, outs, want)
    return dvm.last_launch_variant()["lean"], outs


def _rmsnorm_inputs(rows, cols, seed, shift_elems=0):
    x = wl.randn((rows * cols + 64,), torch.bfloat16, seed).cuda()
    r = wl.randn((rows, cols), torch.bfloat16, seed + 1).cuda()
    w = wl.randn((cols,), torch.bfloat16, seed + 2).cuda()
    xv = x[shift_elems:shift_elems + rows * cols].view(rows, cols)   # (a shifted view: the tensor starts off a 16-byte boundary)
    return [xv, r, w]


def test_dense_aligned_full_rows_and_what_moves_a_program_off_that_build():
    prog = wl.program_add_rmsnorm(4096)
    lean, _ = _run(prog, _rmsnorm_inputs(37, 4096, 1))              # odd row count: the last tile holds one row of two
    assert lean == 7
    lean, _ = _run(prog, _rmsnorm_inputs(37, 4096, 2, shift_elems=3))   # x starts 6 bytes off and its rows fill every slot:
    assert lean == 0                                                    # they wrap around, which only the general interpreter does
    prog2 = wl.program_add_rmsnorm(4000)
    lean, _ = _run(prog2, _rmsnorm_inputs(19, 4000, 3))             # 4000 columns leave slots empty: masks, still aligned
    assert lean == 5
    lean, _ = _run(prog2, _rmsnorm_inputs(19, 4000, 4, shift_elems=3))  # ... and x 6 bytes off: reads are realigned
    assert lean == 4
    prog3 = wl.program_add_rmsnorm(4001)
    lean, _ = _run(prog3, _rmsnorm_inputs(19, 4001, 5))             # rows start off 16-byte boundaries
    assert lean in (0, 3, 4)


def test_row_by_row_copies_aligned_and_not():
    prog = wl.program_masked_softmax(128)
    # the mask's rows are 512 bytes long and fill the slots exactly / 496 bytes: aligned, slots left empty / 500 bytes
    for S, want_lean in ((256, 8), (248, 6), (250, 3)):
        sc = wl.randn((2, 32, S, S), torch.bfloat16, S).cuda()
        m = wl.causal_mask(S, "cuda")
        lean, _ = _run(prog, [sc, m])
        assert lean == want_lean


def test_one_slot_program_aligned_and_not():
    prog = wl.program_if_else_add()
    ins = [wl.randn((7, 33, 1000), torch.float32, 5 + i).cuda() for i in range(4)]
    lean, _ = _run(prog, ins)                                       # one tile slot, three CTAs per SM, every tensor aligned
    v = dvm.last_launch_variant()
    assert lean == 9 and v["single"] == 1 and v["ctas"] == 3
    flat = [wl.randn((7 * 33 * 1000 + 8,), torch.float32, 15 + i).cuda() for i in range(4)]
    ins = [flat[0][1:1 + 7 * 33 * 1000].view(7, 33, 1000)] + [t[:7 * 33 * 1000].view(7, 33, 1000) for t in flat[1:]]
    lean, _ = _run(prog, ins)                                       # the first input starts 4 bytes off: reads are realigned
    assert lean in (0, 1)
    ins = [wl.randn((5, 31, 1001), torch.float32, 25 + i).cuda() for i in range(4)]
    lean, _ = _run(prog, ins)                                       # an odd element count: whichever build, the oracle's result
    assert lean in (0, 1, 9)
