"""GPU parity of programs on VIEWS (Table 1, ViewLoad / ViewStore; dvm_encode_strided): inputs and outputs
given by element strides -- slices, padded rows, permuted outer dims, expanded dims.  The oracle reads the
logical arrays out of the same storage with its own ViewLoad definition, evaluates the program on them, and
writes the expected storage with its ViewStore definition; every element of the storage is compared, so an
element outside the view that the kernel touched shows up."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc
from tests.parity_util import R_TOL, TORCH_DT, gate_errors

pytestmark = pytest.mark.gpu

POISON = -12288.0   # exactly representable in bf16


def _run(prog, in_views, out_views, params=(), tol=None):
    """in_views: (storage tensor, offset, shape, strides) per input; out_views: (storage numel, offset, strides,
    dtype) per output.  Returns the output storages (GPU) after checking them against the oracle."""
    hp = dvm.program_from_nodes(prog.nodes)
    shapes = [tuple(v[2]) for v in in_views]
    code = dvm.encode(hp, shapes, params, in_strides=[list(v[3]) for v in in_views],
                      out_strides=[list(v[2]) for v in out_views])
    dev_in = [v[0].cuda() for v in in_views]
    dev_out = [torch.full((v[0],), POISON, dtype=TORCH_DT[v[3]], device="cuda") for v in out_views]
    es = lambda t: t.element_size()
    ptrs = [t.data_ptr() + v[1] * es(t) for t, v in zip(dev_in, in_views)]
    ptrs += [t.data_ptr() + v[1] * es(t) for t, v in zip(dev_out, out_views)]
    dvm.launch(code, ptrs)
    assert dvm.last_device_status() == 0
    logical = [orc.view_load(wl.to_f64(v[0]), v[1], v[2], v[3]) for v in in_views]
    want = orc.evaluate(prog.nodes, logical, params)
    for k, (v, o) in enumerate(zip(out_views, dev_out)):
        shape = code.out_shapes[k]
        assert tuple(want[k].shape) == tuple(shape)
        exp = orc.view_store(np.full((v[0],), POISON), v[1], shape, v[2], want[k])
        got = wl.to_f64(o)
        idx_touched = exp != POISON
        assert np.array_equal(got[~idx_touched], exp[~idx_touched]), "an element outside the view was written"
        g1, _ = gate_errors(got[idx_touched].reshape(1, -1), exp[idx_touched].reshape(1, -1))
        r = tol if tol is not None else R_TOL[v[3]]
        assert g1 <= r, g1
    return dev_out


def _axpy(dt, rank):
    p = wl.OpProgram("axpy")
    x, y = p.input(dt, rank), p.input(dt, rank)
    p.output(p.binary("add", p.scalar("muls", x, 2.0), y), dt)
    return p


def _dense(shape):
    st, out = 1, []
    for d in reversed(shape):
        out.append(st)
        st *= d
    return out[::-1]


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("B,S,H,D", [(2, 100, 8, 64), (1, 37, 5, 128), (3, 17, 4, 72)])
def test_head_transpose_view(dt, B, S, H, D):
    """x stored [B,S,H,D], read as [B,H,S,D] (the attention head transpose); y and the output dense."""
    x = wl.randn((B * S * H * D,), TORCH_DT[dt], 1)
    y = wl.randn((B * H * S * D,), TORCH_DT[dt], 2)
    shape = (B, H, S, D)
    _run(_axpy(dt, 4), [(x, 0, shape, (S * H * D, D, H * D, 1)), (y, 0, shape, _dense(shape))],
         [(B * H * S * D, 0, _dense(shape), dt)])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_output_into_a_permuted_view(dt):
    """The transpose on the store side: logical [B,H,S,D] written into storage laid out [B,S,H,D]."""
    B, S, H, D = 2, 50, 6, 64
    shape = (B, H, S, D)
    x = wl.randn((B * H * S * D,), TORCH_DT[dt], 3)
    y = wl.randn((B * H * S * D,), TORCH_DT[dt], 4)
    _run(_axpy(dt, 4), [(x, 0, shape, _dense(shape)), (y, 0, shape, _dense(shape))],
         [(B * S * H * D, 0, (S * H * D, D, H * D, 1), dt)])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("R,C,pitch,off", [(300, 74, 100, 3), (64, 1000, 1024, 8), (1, 49, 50, 1), (700, 33, 41, 5)])
def test_column_slices_of_padded_rows(dt, R, C, pitch, off):
    """x[:, off:off+C] of a [R, pitch] buffer in, the result into a column slice of another padded buffer."""
    x = wl.randn((R * pitch,), TORCH_DT[dt], 5)
    y = wl.randn((R * C,), TORCH_DT[dt], 6)
    opitch = pitch + 7
    _run(_axpy(dt, 2), [(x, off, (R, C), (pitch, 1)), (y, 0, (R, C), (C, 1))],
         [(R * opitch, 2, (opitch, 1), dt)])


def test_every_other_row_and_an_expanded_row():
    """x[::2] (row stride 2 C) and a single row expanded over all rows with an explicit stride of 0."""
    R, C = 257, 300
    x = wl.randn((2 * R * C,), torch.float32, 7)
    v = wl.randn((C,), torch.float32, 8)
    _run(_axpy("f32", 2), [(x, 0, (R, C), (2 * C, 1)), (v, 0, (R, C), (0, 1))], [(R * C, 0, (C, 1), "f32")])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_row_reductions_on_a_sliced_view(dt):
    """Softmax over the last dim of scores[:, :, :, :L] (a key-length slice of a padded score buffer)."""
    B, H, S, Lmax, L = 2, 4, 33, 96, 77
    p = wl.OpProgram("softmax")
    x = p.input(dt, 4)
    m = p.reduce("max", x)
    e = p.unary("exp", p.binary("sub", x, m))
    p.output(p.binary("div", e, p.reduce("sum", e)), dt)
    s = wl.randn((B * H * S * Lmax,), TORCH_DT[dt], 9)
    shape = (B, H, S, L)
    _run(p, [(s, 0, shape, (H * S * Lmax, S * Lmax, Lmax, 1))], [(B * H * S * Lmax, 0, (H * S * Lmax, S * Lmax, Lmax, 1), dt)])


def test_view_of_four_outer_dims_that_merge_to_three():
    """[A,B,C,D,E] with a permutation of the outer dims in which two of them stay adjacent and merge."""
    A, B, Cc, D, E = 2, 3, 4, 5, 40
    x = wl.randn((A * B * Cc * D * E,), torch.float32, 10)
    y = wl.randn((A * B * Cc * D * E,), torch.float32, 11)
    shape = (Cc, D, A, B, E)                       # storage [A,B,Cc,D,E] read as [Cc,D,A,B,E]
    xs = (D * E, E, B * Cc * D * E, Cc * D * E, 1)
    _run(_axpy("f32", 5), [(x, 0, shape, xs), (y, 0, shape, _dense(shape))], [(A * B * Cc * D * E, 0, _dense(shape), "f32")])


# ---------------------------------------------------------------- views whose LAST dim is strided (gather / scatter)
@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("R,C", [(5, 7), (64, 100), (257, 333), (3, 4096), (1000, 33)])
def test_transposed_input(dt, R, C):
    """x stored [C,R] read as its transpose [R,C] (column stride R, row stride 1); y and the output dense."""
    x = wl.randn((C * R,), TORCH_DT[dt], 12)
    y = wl.randn((R * C,), TORCH_DT[dt], 13)
    _run(_axpy(dt, 2), [(x, 0, (R, C), (1, R)), (y, 0, (R, C), (C, 1))], [(R * C, 0, (C, 1), dt)])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
@pytest.mark.parametrize("R,C", [(5, 7), (130, 257), (33, 1000)])
def test_transposed_output(dt, R, C):
    """The result written as the transpose: logical [R,C] into storage laid out [C,R]; inputs dense."""
    x = wl.randn((R * C,), TORCH_DT[dt], 14)
    y = wl.randn((R * C,), TORCH_DT[dt], 15)
    _run(_axpy(dt, 2), [(x, 0, (R, C), (C, 1)), (y, 0, (R, C), (C, 1))], [(C * R, 0, (1, R), dt)])


def test_everything_transposed_no_aligned_operand():
    """Both inputs and the output are transposed views: no operand has adjacent columns to align tiles to."""
    R, C = 77, 130
    x = wl.randn((R * C,), torch.float32, 16)
    y = wl.randn((R * C,), torch.float32, 17)
    _run(_axpy("f32", 2), [(x, 0, (R, C), (1, R)), (y, 0, (R, C), (1, R))], [(C * R, 0, (1, R), "f32")])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_column_slice_with_a_step_and_expanded_last_dim(dt):
    """x[:, 1::3] (column stride 3) and a column vector expanded along the last dim with stride 0."""
    R, C = 100, 200
    x = wl.randn((R * (3 * C + 5),), TORCH_DT[dt], 18)
    v = wl.randn((R,), TORCH_DT[dt], 19)
    _run(_axpy(dt, 2), [(x, 1, (R, C), (3 * C + 5, 3)), (v, 0, (R, C), (1, 0))], [(R * C, 0, (C, 1), dt)])


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_softmax_over_a_transposed_view(dt):
    """Row reductions over a gathered operand: softmax along the columns of a [C,R] matrix, written back transposed."""
    R, C = 50, 300
    p = wl.OpProgram("softmax")
    x = p.input(dt, 2)
    m = p.reduce("max", x)
    e = p.unary("exp", p.binary("sub", x, m))
    p.output(p.binary("div", e, p.reduce("sum", e)), dt)
    s = wl.randn((C * R,), TORCH_DT[dt], 20)
    _run(p, [(s, 0, (R, C), (1, R))], [(C * R, 0, (1, R), dt)])


def test_last_two_dims_swapped_in_a_4d_view():
    """[B,H,S,D] read from storage [B,H,D,S] (K^T-style), with a dense second operand."""
    B, H, S, D = 2, 3, 40, 64
    x = wl.randn((B * H * D * S,), torch.float32, 21)
    y = wl.randn((B * H * S * D,), torch.float32, 22)
    shape = (B, H, S, D)
    _run(_axpy("f32", 4), [(x, 0, shape, (H * D * S, D * S, 1, S)), (y, 0, shape, _dense(shape))], [(B * H * S * D, 0, _dense(shape), "f32")])


def _mode_of(code, reg):
    """Layout mode of input register `reg` (local register table of the encoded program)."""
    w = np.frombuffer(code.bytes(), dtype=np.uint32)
    counts = int(w[5])
    lt = 20 + 2 * (counts & 0xff) + 8 * ((counts >> 16) & 0xff)
    return (int(w[lt + reg]) >> 16) & 0xf


@pytest.mark.parametrize("dt,rows,cols,ld,offset", [
    ("bf16", 1000, 777, 1000, 0),      # ragged last row block and column block
    ("bf16", 4096, 512, 4104, 0),      # padded leading dimension (a multiple of 8 elements)
    ("bf16", 640, 300, 640, 3),        # view starts 6 bytes into a 16-byte word: the strips keep that phase
    ("f32", 513, 129, 516, 0),
    ("f32", 2048, 64, 2048, 1),
])
def test_transposed_input_goes_through_strips(dt, rows, cols, ld, offset):
    """x given as the transpose of a [cols, ld] storage (rows adjacent in memory, column stride ld): the tile's
    part of every column is copied as one strip (layout mode 6), not gathered element by element."""
    prog = _axpy(dt, 2)
    tdt = TORCH_DT[dt]
    xs = wl.randn((cols * ld + offset + 8,), tdt, 41)
    ys = wl.randn((rows * cols,), tdt, 42)
    hp = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(hp, [(rows, cols), (rows, cols)], in_strides=[[1, ld], [cols, 1]], out_strides=[[cols, 1]])
    assert _mode_of(code, 0) == 6
    _run(prog, [(xs, offset, (rows, cols), (1, ld)), (ys, 0, (rows, cols), (cols, 1))], [(rows * cols, 0, (cols, 1), dt)])


def test_transposed_batched_and_odd_strides_fall_back():
    """Batched transposes [B, rows, cols] of [B, cols, rows] storage take the strips when the rows per tile divide
    the row count; a column stride that is not a whole number of 16-byte units takes the element gather."""
    prog = _axpy("bf16", 3)
    B, rows, cols = 3, 256, 200
    xs = wl.randn((B * cols * rows,), torch.bfloat16, 43)
    ys = wl.randn((B * rows * cols,), torch.bfloat16, 44)
    _run(prog, [(xs, 0, (B, rows, cols), (cols * rows, 1, rows)), (ys, 0, (B, rows, cols), (rows * cols, cols, 1))],
         [(B * rows * cols, 0, (rows * cols, cols, 1), "bf16")])
    prog2 = _axpy("bf16", 2)
    rows, cols, ld = 300, 100, 301                      # 602 bytes between columns
    xs = wl.randn((cols * ld,), torch.bfloat16, 45)
    ys = wl.randn((rows * cols,), torch.bfloat16, 46)
    hp = dvm.program_from_nodes(prog2.nodes)
    code = dvm.encode(hp, [(rows, cols), (rows, cols)], in_strides=[[1, ld], [cols, 1]], out_strides=[[cols, 1]])
    assert _mode_of(code, 0) == 5
    _run(prog2, [(xs, 0, (rows, cols), (1, ld)), (ys, 0, (rows, cols), (cols, 1))], [(rows * cols, 0, (cols, 1), "bf16")])
