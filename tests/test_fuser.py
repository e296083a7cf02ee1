"""The streaming runtime operator fuser (Sec. 5.2, dynamic graphs): fusion decisions on CPU (no launch), and
fused results against the oracle on the GPU."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc


def _fake_alloc():
    """Result 'buffers' for planning tests: distinct fake addresses, never dereferenced (nothing is flushed)."""
    state = {"next": 0x10000}
    def alloc(shape, dtype):
        state["next"] += 0x100000
        return state["next"]
    return alloc


def test_add_sqrt_is_one_group():
    """The paper's running example: c = a + b, d = sqrt(c) fuse into one meta-kernel (vector-vector pattern)."""
    f = dvm.Fuser(alloc=_fake_alloc())
    a = f.tensor(0x1000, "f32", (37, 100))
    b = f.tensor(0x2000, "f32", (37, 100))
    c = f.binary("add", a, b, (37, 100))
    d = f.unary("sqrt", c, (37, 100))
    assert f.pending() == (2, 1)


def test_independent_chains_stay_separate_and_merge_when_joined():
    f = dvm.Fuser(alloc=_fake_alloc())
    a = f.tensor(0x1000, "f32", (8, 64)); b = f.tensor(0x2000, "f32", (8, 64))
    x = f.tensor(0x3000, "f32", (8, 64)); y = f.tensor(0x4000, "f32", (8, 64))
    c = f.binary("add", a, b, (8, 64))
    z = f.binary("mul", x, y, (8, 64))
    assert f.pending() == (2, 2)              # two independent groups: candidates for spatial stacking
    e = f.binary("sub", c, z, (8, 64))
    assert f.pending() == (3, 1)              # the operator that reads both merges them into one meta-kernel


def test_unfusable_operator_starts_a_new_group():
    """A reduced row cannot be re-expanded over another row length inside one meta-kernel: the operator that
    needs it starts its own group, which reads the first group's result from memory."""
    f = dvm.Fuser(alloc=_fake_alloc())
    a = f.tensor(0x1000, "f32", (16, 300))
    m = f.reduce("max", a, (16, 1))
    w = f.tensor(0x2000, "f32", (16, 500))
    r = f.binary("add", w, m, (16, 500))       # [16,500] + [16,1]: the group of `m` iterates rows of 300
    assert f.pending() == (2, 2)


def test_shape_errors_are_reported_and_leave_the_buffer_intact():
    f = dvm.Fuser(alloc=_fake_alloc())
    a = f.tensor(0x1000, "f32", (4, 10)); b = f.tensor(0x2000, "f32", (4, 11))
    with pytest.raises((dvm.DvmError, AssertionError)):
        f.binary("add", a, b, (4, 10))
    assert f.pending() == (0, 0)


def test_matmul_takes_its_epilogue_on_arrival():
    """Cube-vector fusion (Sec. 5.1) in the stream: a matmul opens a group, the vector operators that arrive behind
    it become its epilogue, and an operator the matmul meta-kernel cannot hold (a second matmul) opens another."""
    f = dvm.Fuser(alloc=_fake_alloc())
    x = f.tensor(0x1000, "bf16", (100, 512)); w = f.tensor(0x100000, "bf16", (512, 256))
    c = f.tensor(0x200000, "bf16", (100, 256))
    mm = f.matmul(x, w, (100, 256))
    assert f.pending() == (1, 1)
    y = f.binary("add", mm, c, (100, 256), "bf16")
    z = f.unary("sigmoid", y, (100, 256), "bf16")
    assert f.pending() == (3, 1)
    w2 = f.tensor(0x300000, "bf16", (256, 64))
    f.matmul(z, w2, (100, 64))                 # its A operand is computed, not in memory: a group of its own
    assert f.pending() == (4, 2)


def test_compare_select_cast_fuse_with_their_producers():
    f = dvm.Fuser(alloc=_fake_alloc())
    a = f.tensor(0x1000, "f32", (9, 70)); b = f.tensor(0x2000, "f32", (9, 70))
    m = f.compare("gt", a, b, (9, 70), "u8")
    s = f.select(m, f.binary("add", a, b, (9, 70)), f.binary("sub", a, b, (9, 70)), (9, 70))
    q = f.cast(f.scalar("muls", s, 10.0, (9, 70)), "i32", (9, 70))
    assert f.pending() == (6, 1)
    with pytest.raises(dvm.DvmError):
        f.select(m, a, 99, (9, 70))            # unknown value id
    assert f.pending() == (6, 1)


# ------------------------------------------------------------------------------------------- on the GPU
def _oracle_chain(nodes_fn, ins, out_dtypes=None):
    p = wl.OpProgram("chain")
    ids = [p.input("bf16" if t.dtype == torch.bfloat16 else "f32", t.dim()) for t in ins]
    outs = nodes_fn(p, ids)
    for k, o in enumerate(outs):
        p.output(o, out_dtypes[k] if out_dtypes else "f32")
    return orc.evaluate(p.nodes, [wl.to_f64(t) for t in ins])


def _close(got, want, r=1e-5):
    """Gate G1 of the parity tests: |g - o| <= r * max(|o|, row max |o|), every element."""
    g = wl.to_f64(got)
    assert g.shape == want.shape
    den = np.maximum(np.abs(want), np.max(np.abs(want), axis=-1, keepdims=True))
    err = np.abs(g - want)
    assert np.all(err <= r * den), float(np.max(err / np.maximum(den, 1e-300)))


@pytest.mark.gpu
def test_softmax_like_stream_matches_oracle_and_elides_intermediates():
    x = wl.randn((64, 1000), torch.float32, 1).cuda()
    f = dvm.Fuser()
    vx = f.tensor(x)
    m = f.reduce("max", vx, (64, 1))
    d = f.binary("sub", vx, m, (64, 1000))
    e = f.unary("exp", d, (64, 1000))
    s = f.reduce("sum", e, (64, 1))
    y = f.binary("div", e, s, (64, 1000))
    for v in (m, d, e, s):
        f.release(v)                       # the framework keeps only y
    assert f.pending() == (5, 1)
    f.flush()
    torch.cuda.synchronize()
    st = f.stats()
    assert st["groups"] == 1 and st["launches"] == 1 and st["stores_elided"] == 4
    want = _oracle_chain(lambda p, i: [p.binary("div", p.unary("exp", p.binary("sub", i[0], p.reduce("max", i[0]))),
                                                p.reduce("sum", p.unary("exp", p.binary("sub", i[0], p.reduce("max", i[0])))))], [x])[0]
    got = wl.to_f64(f.tensors[y])
    assert np.max(np.abs(got - want)) <= 1e-5 * np.max(np.abs(want))


@pytest.mark.gpu
@pytest.mark.parametrize("temporal", [True, False])
def test_independent_groups_run_as_one_stacked_launch_and_dependents_later(temporal):
    a = wl.randn((100, 333), torch.float32, 1).cuda(); b = wl.randn((100, 333), torch.float32, 2).cuda()
    x = wl.randn((7, 4000), torch.float32, 3).cuda()
    w = wl.randn((100, 64), torch.float32, 4).cuda()
    f = dvm.Fuser(temporal_stacking=temporal)
    va, vb, vx, vw = f.tensor(a), f.tensor(b), f.tensor(x), f.tensor(w)
    c = f.unary("sqrt", f.unary("abs", f.binary("add", va, vb, (100, 333)), (100, 333)), (100, 333))   # group 1
    z = f.scalar("muls", f.unary("sigmoid", vx, (7, 4000)), 3.0, (7, 4000))                                # group 2
    m = f.reduce("max", c, (100, 1))                                                                      # joins group 1
    r = f.binary("mul", vw, m, (100, 64))                       # rows of 64 against a [100,1]: its own group, one level up
    assert f.pending() == (7, 3)
    n0 = dvm.launch_count()
    f.flush()
    torch.cuda.synchronize()
    # level 0: groups 1 and 2, stacked; level 1: the dependent group -- in the same launch behind an in-kernel
    # wait (temporal stacking), or in a second launch on the stream
    assert dvm.launch_count() - n0 == (1 if temporal else 2)
    assert dvm.last_device_status() == 0
    # against the oracle: the four kept values as outputs of the same operator chain, evaluated in fp64
    def chain(p, i):
        pc = p.unary("sqrt", p.unary("abs", p.binary("add", i[0], i[1])))
        pm = p.reduce("max", pc)
        return [pc, p.scalar("muls", p.unary("sigmoid", i[2]), 3.0), pm, p.binary("mul", i[3], pm)]
    want = _oracle_chain(chain, [a, b, x, w])
    for v, o in zip((c, z, m, r), want):
        _close(f.tensors[v], o)
    # the row maximum picks one stored element of c: bit-exact against the device's own c
    cc = f.tensors[c]
    assert torch.equal(f.tensors[m], cc.max(dim=1, keepdim=True).values)
    # second check, library routine on the device
    assert torch.allclose(cc, torch.sqrt((a + b).abs()), rtol=1e-6, atol=0)


@pytest.mark.gpu
def test_values_survive_a_flush_and_feed_later_operators():
    a = wl.randn((33, 257), torch.float32, 5).cuda()
    f = dvm.Fuser()
    va = f.tensor(a)
    c = f.scalar("adds", va, 1.5, (33, 257))
    f.flush()
    d = f.binary("mul", c, va, (33, 257))     # c now lies in memory
    f.flush()
    torch.cuda.synchronize()
    want = _oracle_chain(lambda p, i: [p.binary("mul", p.scalar("adds", i[0], 1.5), i[0])], [a])[0]
    _close(f.tensors[d], want)
    assert torch.allclose(f.tensors[d], (a + 1.5) * a, rtol=1e-6, atol=0)   # second check
    assert f.stats()["launches"] == 2


@pytest.mark.gpu
def test_long_levels_keep_their_own_launches():
    """Dependent groups whose levels exceed 1024 tiles are not stacked temporally: one launch per level."""
    R, C = 3000, 4096                      # 3000 tiles of 256 x 16 elements per level
    a = wl.randn((R, C), torch.float32, 6).cuda()
    w = wl.randn((R, 64), torch.float32, 7).cuda()
    f = dvm.Fuser()
    va, vw = f.tensor(a), f.tensor(w)
    m = f.reduce("max", f.unary("abs", va, (R, C)), (R, 1))
    r = f.binary("mul", vw, m, (R, 64))    # rows of 64 against [R,1]: a second group, one level up
    n0 = dvm.launch_count()
    f.flush()
    torch.cuda.synchronize()
    assert dvm.launch_count() - n0 == 2
    assert dvm.last_device_status() == 0
    def chain(p, i):
        pm = p.reduce("max", p.unary("abs", i[0]))
        return [pm, p.binary("mul", i[1], pm)]
    want = _oracle_chain(chain, [a, w])
    # |x| and max are exact in any precision: the maxima equal the oracle's bit for bit
    assert np.array_equal(wl.to_f64(f.tensors[m]), want[0])
    _close(f.tensors[r], want[1])


@pytest.mark.gpu
def test_if_else_add_stream_with_mask_and_quantised_output():
    """Table 1 Cmp / Select / Cast through the streaming fuser: one group, one launch; the u8 mask and the i32
    codes bit-exact against the oracle (inputs on a grid of sixteenths, so every decision is exact in fp32)."""
    a = (torch.round(wl.randn((77, 1500), torch.float32, 11) * 16) / 16).cuda()
    b = (torch.round(wl.randn((77, 1500), torch.float32, 12) * 16) / 16).cuda()
    f = dvm.Fuser()
    va, vb = f.tensor(a), f.tensor(b)
    m = f.compare("gt", va, vb, a.shape, "u8")
    s = f.select(m, f.binary("add", va, vb, a.shape), f.binary("sub", va, vb, a.shape), a.shape)
    q = f.cast(f.scalar("muls", s, 4.0, a.shape), "i32", a.shape)
    assert f.pending() == (6, 1)
    n0 = dvm.launch_count()
    f.flush()
    torch.cuda.synchronize()
    assert dvm.launch_count() - n0 == 1 and dvm.last_device_status() == 0
    def chain(p, i):
        pm = p.compare("gt", i[0], i[1])
        ps = p.select(pm, p.binary("add", i[0], i[1]), p.binary("sub", i[0], i[1]))
        return [pm, ps, p.cast(p.scalar("muls", ps, 4.0), "i32")]
    want = _oracle_chain(chain, [a, b], ["u8", "f32", "i32"])
    assert f.tensors[m].dtype == torch.uint8 and f.tensors[q].dtype == torch.int32
    assert np.array_equal(f.tensors[m].cpu().numpy().astype(np.float64), want[0])
    assert np.array_equal(wl.to_f64(f.tensors[s]), want[1])
    assert np.array_equal(f.tensors[q].cpu().numpy().astype(np.float64), want[2])


@pytest.mark.gpu
def test_matmul_with_streamed_epilogue_matches_oracle_in_one_launch():
    M, K, N = 300, 512, 384
    x = wl.randn((M, K), torch.bfloat16, 21).cuda()
    w = wl.randn((K, N), torch.bfloat16, 22, std=K ** -0.5).cuda()
    c = wl.randn((M, N), torch.bfloat16, 23).cuda()
    f = dvm.Fuser()
    vx, vw, vc = f.tensor(x), f.tensor(w), f.tensor(c)
    mm = f.matmul(vx, vw, (M, N))
    y = f.unary("sigmoid", f.binary("add", mm, vc, (M, N), "bf16"), (M, N), "f32")
    f.release(mm)
    assert f.pending() == (3, 1)
    n0 = dvm.launch_count()
    f.flush()
    torch.cuda.synchronize()
    assert dvm.launch_count() - n0 == 1 and dvm.last_device_status() == 0
    want = _oracle_chain(lambda p, i: [p.unary("sigmoid", p.binary("add", p.matmul(i[0], i[1]), i[2]))], [x, w, c])[0]
    # fp32 accumulation over K = 512 products of bf16 values, then sigmoid (slope <= 1/4)
    assert np.max(np.abs(wl.to_f64(f.tensors[y]) - want)) <= 2e-5
    # a matmul next to an independent vector group: the stacked launch refuses the mix, each runs by itself
    f2 = dvm.Fuser()
    vx, vw, vc = f2.tensor(x), f2.tensor(w), f2.tensor(c)
    mm = f2.matmul(vx, vw, (M, N), "f32")
    e = f2.unary("exp", vc, (M, N))
    assert f2.pending() == (2, 2)
    f2.flush()
    torch.cuda.synchronize()
    assert dvm.last_device_status() == 0
    want = _oracle_chain(lambda p, i: [p.matmul(i[0], i[1]), p.unary("exp", i[2])], [x, w, c])
    assert np.max(np.abs(wl.to_f64(f2.tensors[mm]) - want[0])) <= 1e-4 * np.max(np.abs(want[0]))
    _close(f2.tensors[e], want[1])


@pytest.mark.gpu
def test_two_reduced_axes_split_into_two_levels():
    """A column statistic followed by a row normalisation: one meta-kernel reduces over one axis, so the chain
    becomes two groups on consecutive levels; both results against the oracle."""
    a = wl.randn((300, 257), torch.float32, 31).cuda()
    f = dvm.Fuser()
    va = f.tensor(a)
    cm = f.reduce("max", f.unary("abs", va, a.shape), (1, 257), axis=-2)      # column maxima of |a|
    sc = f.binary("div", va, cm, a.shape)                                     # a scaled column by column
    rs = f.reduce("sum", f.binary("mul", sc, sc, a.shape), (300, 1))          # row sums of squares
    out = f.binary("div", sc, f.unary("sqrt", rs, (300, 1)), a.shape)
    ops, groups = f.pending()
    assert ops == 7 and groups >= 2
    f.flush()
    torch.cuda.synchronize()
    assert dvm.last_device_status() == 0
    def chain(p, i):
        pc = p.reduce("max", p.unary("abs", i[0]), axis=-2)
        ps = p.binary("div", i[0], pc)
        pr = p.reduce("sum", p.binary("mul", ps, ps))
        return [pc, p.binary("div", ps, p.unary("sqrt", pr))]
    want = _oracle_chain(chain, [a])
    assert np.array_equal(wl.to_f64(f.tensors[cm]), want[0])                  # |x| and max are exact
    _close(f.tensors[out], want[1])
