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


# ------------------------------------------------------------------------------------------- on the GPU
def _oracle_chain(nodes_fn, ins):
    p = wl.OpProgram("chain")
    ids = [p.input("f32", t.dim()) for t in ins]
    outs = nodes_fn(p, ids)
    for o in outs:
        p.output(o, "f32")
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
