"""Host logic on CPU: the C-ABI library loads and exports every declared symbol, the paper's
tiling example and tile partition, encoder geometry, verifier and dump."""
import ctypes
import os
import re

import numpy as np

import pytest

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from paper_2603_24239_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "dvm.h")).read() + open(os.path.join(ROOT, "include", "dvm_fuser.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(dvm_[a-z0-9_]+)\s*\(", hdr))
    assert len(declared) >= 25
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"libdvm.so does not export {name}"
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)


def test_paper_tiling_example():
    """Sec. 4.2 worked example: fp16 [32,1024] add, 40 cores, 32-byte instruction width."""
    row = [l for l in open(os.path.join(ROOT, "tests", "golden", "paper_tiling_example.txt"))
           if not l.startswith("#")][0].split()
    total, cores, align_b, esize, want_t, want_n, want_tail, want_r = map(int, row)
    r = dvm.hardware_align_div(total, cores, align_b // esize, 1 << 20, 2)
    assert r == {"min_cost_tile": want_t, "rounded_tile": want_r, "n_tiles": want_n, "tail": want_tail}
    # the minimum is unique: brute force over every tile size
    costs = {t: -(-(-(-total // t)) // cores) * (t + 2) for t in range(1, total + 1)}
    best = min(costs.values())
    assert [t for t, c in costs.items() if c == best] == [want_t]
    # rounding never exceeds the tile size limit
    r = dvm.hardware_align_div(total, cores, 16, 825, 2)
    assert r["rounded_tile"] <= 825


@pytest.mark.parametrize("M,N", [(41, 40), (40, 40), (1, 40), (0, 7), (1000, 148), (7, 444)])
def test_vm_tile_partition_is_exact_cover(M, N):
    """Algorithm 2: core id runs [m*id, min(M, m*(id+1))), m = ceil(M/N)."""
    seen = []
    busy = 0
    for i in range(N):
        b, e = dvm.vm_tile_range(M, N, i)
        seen += list(range(b, e))
        busy += e > b
    assert seen == list(range(M))
    if (M, N) == (41, 40):
        assert busy == 21 and dvm.vm_tile_range(M, N, 20) == (40, 41)


def _enc(prog, shapes, params=()):
    return dvm.encode(dvm.program_from_nodes(prog.nodes), shapes, params)


def test_encode_geometry_and_shapes():
    c = _enc(wl.program_add_rmsnorm(), [(1000, 4096), (1000, 4096), (4096,)])
    assert c.out_shapes == [(1000, 4096), (1000, 4096)]
    info = dvm.code_info(c)
    # 4096 columns: 64 threads x 64 elements (four rows per tile), 128 x 32 or 256 x 16
    assert info["threads_per_row"] in (64, 128, 256) and info["vector_width"] == 8
    assert info["n_tiles"] == 1000 * info["threads_per_row"] // 256
    assert info["kernel_type"] == 1 and info["n_tile_regs"] == 3   # three inputs in local registers, no temporaries
    c = _enc(wl.program_masked_softmax(), [(2, 32, 100, 100), (1, 1, 100, 100)])
    assert c.out_shapes == [(2, 32, 100, 100)]
    info = dvm.code_info(c)
    assert info["threads_per_row"] * 64 >= 100                # rows of 100 bf16 start on 8-byte boundaries only
    assert info["n_tiles"] == -(-6400 // (256 // info["threads_per_row"]))
    # pure elementwise program collapses to a flat range
    c = _enc(wl.program_c1(), [(7, 1531)] * 3)
    d = dvm.disassemble(c)
    assert "flags=A-F" in d and "exp" in d and "block_dim=" in d and "body_tile=" in d
    # zero-size instance
    c = _enc(wl.program_c1(), [(0, 5)] * 3)
    assert dvm.code_info(c)["n_tiles"] == 0 and c.out_shapes == [(0, 5)]


def test_encode_is_shape_dependent_and_deterministic():
    p = dvm.program_from_nodes(wl.program_layernorm().nodes)
    a = dvm.encode(p, [(10, 100)], (0.01,)).bytes()
    b = dvm.encode(p, [(10, 100)], (0.01,)).bytes()
    c = dvm.encode(p, [(11, 100)], (0.01,)).bytes()
    assert a == b and a != c


def test_encode_errors():
    p = dvm.program_from_nodes(wl.program_c1().nodes)
    with pytest.raises(dvm.DvmError) as e:
        dvm.encode(p, [(7, 5), (7, 6), (7, 5)])
    assert e.value.status == -2
    with pytest.raises(dvm.DvmError) as e:
        dvm.encode(p, [(7, 5), (7, 5)])
    assert e.value.status == -1
    # a reduced row longer than a tile runs in phases; nine reductions that each need the one before would
    # need nine phases and nine per-row scalars that outlive their tiles: more than the machine holds
    q = dvm.program_from_nodes(wl.program_layernorm().nodes)
    assert dvm.verify(dvm.encode(q, [(4, 17000)], (1 / 17000,))) == 0
    deep = wl.OpProgram("deep")
    v = deep.input("f32", 2)
    for _ in range(9):
        v = deep.binary("sub", v, deep.reduce("max", v))
    deep.output(v, "f32")
    assert dvm.verify(dvm.encode(dvm.program_from_nodes(deep.nodes), [(4, 8000)])) == 0
    with pytest.raises(dvm.DvmError) as e:
        dvm.encode(dvm.program_from_nodes(deep.nodes), [(4, 17000)])
    assert e.value.status == -3
    # missing runtime scalar
    with pytest.raises(dvm.DvmError):
        dvm.encode(q, [(4, 50)], ())
    # unfinalized program
    r = dvm.Program(); r.input("f32", 1)
    with pytest.raises(dvm.DvmError):
        dvm.encode(r, [(4,)])


def test_buffer_too_small_reports_need():
    import ctypes as C
    p = dvm.program_from_nodes(wl.program_c1().nodes)
    enc = binding.Encoder(p)
    need = enc.encode([(7, 1531)] * 3)
    small = (C.c_uint64 * 4)()
    size = C.c_size_t(0)
    st = binding.lib.dvm_encode(p._h, enc.shapes, 3, enc.scalars, 0, small, 32, C.byref(size), None, 0)
    assert st == -4 and size.value == need


def test_verify_rejects_malformed_code():
    c = _enc(wl.program_masked_softmax(), [(1, 2, 40, 40), (1, 1, 40, 40)])
    good = bytearray(c.bytes())
    assert dvm.verify(bytes(good)) == 0
    import random
    rnd = random.Random(7)
    rejected = 0
    for _ in range(400):
        bad = bytearray(good)
        k = rnd.randrange(len(bad))
        bad[k] ^= 1 << rnd.randrange(8)
        st = dvm.verify(bytes(bad))
        assert st in (0, -5)
        rejected += st == -5
    assert rejected > 100           # most single-bit flips are caught; the rest are value changes
    assert dvm.verify(bytes(good[:-4])) == -5
    assert dvm.verify(b"\0" * 80) == -5
    bad = bytearray(good); bad[-4] = 0xEE     # unknown instruction id in the last word
    assert dvm.verify(bytes(bad)) == -5


def test_local_register_pressure():
    p = wl.OpProgram("wide")
    ins = [p.input("f32", 2) for _ in range(6)]
    acc = p.binary("mul", ins[0], ins[1])
    for i in range(2, 6):
        acc = p.binary("add", acc, ins[i])
    for i in range(6):                     # every input is used again at the end
        acc = p.binary("mul", acc, ins[i])
    p.output(acc, "f32")
    c = _enc(p, [(3, 50)] * 6)
    assert dvm.code_info(c)["n_tile_regs"] == 6          # inputs stay in their local registers, no spill
    q = wl.OpProgram("too_wide")
    ins = [q.input("f32", 2) for _ in range(10)]
    acc = q.binary("mul", ins[0], ins[1])
    for i in range(2, 10):
        acc = q.binary("add", acc, ins[i])
    for i in range(10):
        acc = q.binary("mul", acc, ins[i])
    q.output(acc, "f32")
    with pytest.raises(dvm.DvmError) as e:
        _enc(q, [(3, 50)] * 10)
    assert e.value.status == -3


def test_encode_latency_budget():
    """Host encode stays far below the 50 us budget even on this CPU machine (median over many calls)."""
    import time
    p = dvm.program_from_nodes(wl.program_add_rmsnorm().nodes)
    enc = binding.Encoder(p)
    ts = []
    for i in range(2000):
        t0 = time.perf_counter_ns()
        enc.encode(((1000 + i, 4096), (1000 + i, 4096), (4096,)))
        ts.append(time.perf_counter_ns() - t0)
    ts.sort()
    assert ts[len(ts) // 2] < 50_000


def test_encode_batch_matches_single_encodes():
    """dvm_encode_batch produces, instance by instance, the bytes dvm_encode produces."""
    from paper_2603_24239_b200 import binding
    dvm.set_elems_per_thread(16)
    try:
        items = [("gelu_affine", 3, 65), ("layernorm", 17, 100), ("sigmoid_mul", 1, 64), ("layernorm", 512, 4096)]
        progs = [dvm.program_from_nodes(wl.stack_program(k).nodes) for k, _, _ in items]
        shapes = [{"gelu_affine": [(r, c), (1, c), (1, c)], "layernorm": [(r, c)], "sigmoid_mul": [(r, c), (r, c)]}[k]
                  for k, r, c in items]
        scalars = [[1.0 / c] if k == "layernorm" else [] for k, r, c in items]
        be = binding.BatchEncoder(progs)
        be.encode(shapes, scalars)
        for i, p in enumerate(progs):
            single = dvm.encode(p, shapes[i], scalars[i])
            assert bytes(be.bufs[i])[: be.sizes[i]] == single.bytes()
        # a failing instance is reported with its index
        bad = [list(s) for s in shapes]
        bad[2] = [(1, 64), (2, 63)]
        with pytest.raises(dvm.DvmError) as ei:
            be.encode(bad, scalars)
        assert "instance 2" in str(ei.value)
    finally:
        dvm.set_elems_per_thread(0)


def test_stacked_levels_rejects_decreasing_levels_before_any_launch():
    """dvm_launch_stacked_levels: levels must be non-decreasing (the work queue hands tiles out in that
    order); the check is on the host, ahead of every CUDA call."""
    p = wl.OpProgram("add")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("add", a, b), "f32")
    hp = dvm.program_from_nodes(p.nodes)
    codes = [dvm.encode(hp, [(4, 8), (4, 8)]) for _ in range(2)]
    fake = [[0x1000, 0x2000, 0x3000], [0x3000, 0x2000, 0x4000]]   # never dereferenced: the call fails first
    with pytest.raises(dvm.DvmError) as ei:
        dvm.launch_stacked(codes, fake, levels=[1, 0])
    assert ei.value.status == -1   # DVM_ERR_INVALID_ARG


def test_min_resident_ctas_picks_a_geometry_that_fits_twice_per_sm():
    """A wide GELU(x*w+b) row at 16 elements per thread: unconstrained, one row per tile with whole-row images
    of w and b (195 units per slot: one CTA per SM; the fused activation needs no temporary); with
    dvm_set_min_resident_ctas(2), column blocks that fit twice per SM, chosen by total work (the program shares
    its launch: no waves of its own to fill)."""
    p = dvm.program_from_nodes(wl.stack_program("gelu_affine").nodes)
    shapes = [(148, 2893), (1, 2893), (1, 2893)]
    dvm.set_elems_per_thread(16)
    try:
        free = dvm.disassemble(dvm.encode(p, shapes))
        dvm.set_min_resident_ctas(2)
        tight = dvm.disassemble(dvm.encode(p, shapes))
    finally:
        dvm.set_min_resident_ctas(0)
        dvm.set_elems_per_thread(0)
    assert "local_units=195" in free and "col_blocks=1 " in free and "gelu" in free
    # costed by total work: 3 column blocks of 1020 columns waste fewer slots than 2 of 2044 (2893 = 2 x 1020 + 853)
    assert "local_units=99" in tight and "col_blocks=3 " in tight and "threads_per_row=64" in tight


def test_encode_strided_views_geometry_and_errors():
    """dvm_encode_strided: the caller's element strides reach the operand descriptors; rows must be adjacent
    in memory; a stored view must address every element once."""
    p = wl.OpProgram("axpy")
    x, y = p.input("f32", 4), p.input("f32", 4)
    p.output(p.binary("add", p.scalar("muls", x, 2.0), y), "f32")
    hp = dvm.program_from_nodes(p.nodes)
    B, S, H, D = 2, 100, 8, 64
    shape = (B, H, S, D)
    text = dvm.disassemble(dvm.encode(hp, [shape, shape], in_strides=[[S * H * D, D, H * D, 1], None]))
    assert "in0 f32 col_stride=1 strides=[512,64,51200]" in text      # S, H, B over storage [B,S,H,D]
    assert "in1 f32 col_stride=1 strides=[64,6400,51200]" in text     # dense [B,H,S,D]
    # all-dense strides give the bytes of the plain encode
    dense = [H * S * D, S * D, D, 1]
    assert dvm.encode(hp, [shape, shape], in_strides=[dense, dense], out_strides=[dense]).bytes() == \
        dvm.encode(hp, [shape, shape]).bytes()
    # a strided last dim is gathered: its column stride reaches the descriptor, the register holds fp32
    text = dvm.disassemble(dvm.encode(hp, [shape, shape], in_strides=[[S * H * D, D, 1, H], None]))
    assert "in0 f32 col_stride=8 strides=[1,64,51200]" in text
    for kwargs, status in [(dict(in_strides=[[-1, 1, 1, 1], None]), -1),               # negative stride
                           (dict(out_strides=[[S * H * D, D, D, 1]]), -1),             # two rows at one address
                           (dict(out_strides=[[H * S * D, S * D, 0, 1]]), -1)]:        # zero stride in an output
        with pytest.raises(dvm.DvmError) as ei:
            dvm.encode(hp, [shape, shape], **kwargs)
        assert ei.value.status == status, kwargs
    # an expanded input (stride 0) is a broadcast
    text = dvm.disassemble(dvm.encode(hp, [shape, shape], in_strides=[[0, 0, 0, 1], None]))
    assert "in0 f32 col_stride=1 strides=[0,0,0]" in text


def test_pow_and_isfinite_encode_for_the_extended_variant():
    p = wl.OpProgram("pow")
    a, b = p.input("f32", 2), p.input("f32", 2)
    p.output(p.unary("isfinite", p.binary("pow", a, b)), "f32")
    text = dvm.disassemble(dvm.encode(dvm.program_from_nodes(p.nodes), [(5, 100), (5, 100)]))
    assert "pow " in text and "isfinite" in text
    # Pow takes tile operands: a per-row value as exponent is refused
    q = wl.OpProgram("pow_row")
    a = q.input("f32", 2)
    q.output(q.binary("pow", a, q.reduce("max", a)), "f32")
    with pytest.raises(dvm.DvmError) as ei:
        dvm.encode(dvm.program_from_nodes(q.nodes), [(5, 100)])
    assert ei.value.status == -3


def test_reduce_over_another_axis_is_lowered_to_views():
    """Sum over axis -2 of [M, S, N]: encoded as a last-axis reduction over the permuted view (the reduced axis
    becomes the column dim with its memory stride N); output shape reported in the caller's order."""
    p = wl.OpProgram("r")
    a = p.input("f32", 3)
    s1 = p.reduce("sum", a, -2)
    p.output(p.binary("sub", a, s1), "f32")         # the reduced value is used: the view lowering
    hp = dvm.program_from_nodes(p.nodes)
    code = dvm.encode(hp, [(4, 50, 8)])
    assert code.out_shapes[0] == (4, 50, 8)
    text = dvm.disassemble(code)
    assert "cols=50 " in text and "in0 f32 col_stride=8" in text and "rowsum" in text
    # a reduction that is a result only: the tiles keep their natural shape (columns adjacent in memory) and
    # combine their rows into the fp32 result atomically -- the stored view has stride 0 along the reduced axis
    r = wl.OpProgram("r2")
    a = r.input("f32", 3)
    r.output(r.reduce("max", r.unary("abs", a), -2), "f32")
    code = dvm.encode(dvm.program_from_nodes(r.nodes), [(4, 50, 256)])
    assert code.out_shapes[0] == (4, 1, 256)
    text = dvm.disassemble(code)
    assert "cols=256 " in text and "strides=[0,256,0] combine=max" in text and "rowmax" not in text
    # ... but not into a bf16 result (the view lowering again)
    r = wl.OpProgram("r3")
    a = r.input("bf16", 3)
    r.output(r.reduce("sum", a, -2), "bf16")
    assert "combine" not in dvm.disassemble(dvm.encode(dvm.program_from_nodes(r.nodes), [(4, 50, 256)]))
    # two different reduced axes in one program, or a last-axis reduce next to another axis: refused
    q = wl.OpProgram("rr")
    a = q.input("f32", 3)
    q.output(q.binary("add", q.reduce("sum", a, -2), q.reduce("sum", a, -3)), "f32")
    with pytest.raises(dvm.DvmError) as ei:
        dvm.encode(dvm.program_from_nodes(q.nodes), [(4, 5, 8)])
    assert ei.value.status == -3
    r1 = wl.OpProgram("r1")                      # axis -2 of a rank-1 value: no such axis
    a = r1.input("f32", 1)
    r1.output(r1.reduce("sum", a, -2), "f32")
    with pytest.raises(dvm.DvmError) as ei:
        dvm.encode(dvm.program_from_nodes(r1.nodes), [(9,)])
    assert ei.value.status == -1


def test_single_slot_hint_only_where_it_buys_a_second_cta():
    """if-else-add at 16 elements per thread: 388 units per slot -- two slots fit once per SM, one slot twice:
    the header carries the single-slot hint.  A program that fits twice with two slots does not, and neither
    does any program encoded for a stacked launch (dvm_set_min_resident_ctas(2): its CTAs keep two slots)."""
    flag = lambda code: (int(np.frombuffer(code.bytes(), dtype=np.uint32)[6]) >> 24) & 128
    ifelse = dvm.program_from_nodes(wl.program_if_else_add().nodes)
    assert flag(dvm.encode(ifelse, [(8, 64, 4096)] * 4))
    norm = dvm.program_from_nodes(wl.program_add_rmsnorm().nodes)
    assert not flag(dvm.encode(norm, [(300, 4096), (300, 4096), (4096,)]))
    dvm.set_min_resident_ctas(2)
    try:
        assert not flag(dvm.encode(ifelse, [(8, 64, 4096)] * 4))
    finally:
        dvm.set_min_resident_ctas(0)


def test_encoder_knobs_are_per_thread():
    """dvm_set_elems_per_thread / dvm_set_min_resident_ctas / dvm_set_num_cores act on the calling thread only."""
    import threading
    lib = dvm.binding.lib
    seen = {}

    def worker():
        lib.dvm_set_elems_per_thread(16)
        lib.dvm_set_min_resident_ctas(2)
        lib.dvm_set_num_cores(10)
        seen["inside"] = (lib.dvm_get_elems_per_thread(), lib.dvm_get_min_resident_ctas(), lib.dvm_get_num_cores())

    t = threading.Thread(target=worker)
    t.start()
    t.join()
    assert seen["inside"] == (16, 2, 10)
    assert (lib.dvm_get_elems_per_thread(), lib.dvm_get_min_resident_ctas(), lib.dvm_get_num_cores()) == (0, 0, 444)
