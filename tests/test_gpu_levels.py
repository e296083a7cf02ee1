"""GPU parity of temporal stacking of DEPENDENT programs (dvm_launch_stacked_levels): programs of a later
level read, inside the same kernel, what programs of earlier levels store.  The oracle runs the programs one
after the other on the CPU."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import gate_errors, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[16, 32])
def elems_per_thread(request):
    dvm.set_elems_per_thread(request.param)
    yield request.param
    dvm.set_elems_per_thread(0)


def _binary(op, rank=2):
    p = wl.OpProgram(op)
    a, b = p.input("f32", rank), p.input("f32", rank)
    p.output(p.binary(op, a, b), "f32")
    return p


def _scale_tanh():
    p = wl.OpProgram("scale_tanh")
    a = p.input("f32", 2)
    p.output(p.unary("tanh", p.scalar("muls", a, 0.5)), "f32")
    return p


def _row_norm():
    """y = x / sqrt(sum(x^2) + 1): one row reduction, the row scalar applied to the row."""
    p = wl.OpProgram("row_norm")
    x = p.input("f32", 2)
    ms = p.scalar("adds", p.reduce("sum", p.binary("mul", x, x)), 1.0)
    p.output(p.binary("mul", x, p.unary("rsqrt", ms)), "f32")
    return p


def _run_dag(R, C, seed, repeats=1):
    """level 0: t0 = a + b, t1 = tanh(0.5 c); level 1: t2 = t0 * t1, t3 = row_norm(t0); level 2: t4 = t2 - t3."""
    a, b, c = (wl.randn((R, C), torch.float32, seed + k) for k in range(3))
    progs = [(_binary("add"), [0, 1], 0), (_scale_tanh(), [2], 0), (_binary("mul"), [3, 4], 1), (_row_norm(), [3], 1),
             (_binary("sub"), [5, 6], 2)]
    host = [a, b, c]       # values 0..2 are the inputs, 3.. the programs' results in order
    for prog, ins, _ in progs:
        want = oracle_run(prog, [host[i] for i in ins])
        host.append(torch.from_numpy(want[0]))   # fp64: the oracle chain is exact in between
    dev = [t.cuda() for t in (a, b, c)]
    dev += [torch.full((R, C), float("nan"), dtype=torch.float32, device="cuda") for _ in progs]
    codes, tls, levels = [], [], []
    for k, (prog, ins, lv) in enumerate(progs):
        codes.append(dvm.encode(dvm.program_from_nodes(prog.nodes), [(R, C)] * len(ins)))
        tls.append([dev[i] for i in ins] + [dev[3 + k]])
        levels.append(lv)
    for _ in range(repeats):
        for t in dev[3:]:
            t.fill_(float("nan"))
        n0 = dvm.launch_count()
        dvm.launch_stacked(codes, tls, levels=levels)
        assert dvm.last_device_status() == 0
        assert dvm.launch_count() - n0 == 1
        for k in range(len(progs)):
            g1, _ = gate_errors(wl.to_f64(dev[3 + k]), host[3 + k].numpy())
            assert g1 <= 3e-5, (k, g1)   # three fp32 programs deep: each adds at most 1e-5 row-scaled


@pytest.mark.parametrize("R,C", [(1, 7), (5, 100), (300, 333), (1024, 2048), (40000, 64), (3, 4096)])
def test_dag_of_five_programs_in_one_launch(R, C):
    """From launches with fewer tiles than resident CTAs (every first tile of a later level is held back) to
    launches where CTAs cross the level boundaries in mid-queue."""
    _run_dag(R, C, seed=R + C)


def test_levels_launch_leaves_the_counters_at_rest():
    """Repeated launches through the same queue slots: the completion counter is back at zero each time."""
    _run_dag(2000, 512, seed=9, repeats=6)


def test_long_chain_of_levels():
    """x_{k+1} = x_k * 1.01 + y, 24 levels deep, one program per level: every tile of level k+1 waits for level k."""
    R, C = 700, 300
    p = wl.OpProgram("axpy")
    x, y = p.input("f32", 2), p.input("f32", 2)
    p.output(p.binary("add", p.scalar("muls", x, 1.01), y), "f32")
    n = 24
    x0, yy = wl.randn((R, C), torch.float32, 1), wl.randn((R, C), torch.float32, 2)
    bufs = [x0.cuda()] + [torch.full((R, C), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n)]
    ydev = yy.cuda()
    hp = dvm.program_from_nodes(p.nodes)
    codes = [dvm.encode(hp, [(R, C), (R, C)]) for _ in range(n)]
    tls = [[bufs[k], ydev, bufs[k + 1]] for k in range(n)]
    dvm.launch_stacked(codes, tls, levels=list(range(n)))
    assert dvm.last_device_status() == 0
    want = wl.to_f64(x0)
    for k in range(n):
        want = oracle_run(p, [torch.from_numpy(want), yy])[0]
    g1, _ = gate_errors(wl.to_f64(bufs[n]), want)
    assert g1 <= n * 1e-5, g1


def test_same_level_everywhere_equals_plain_stacking():
    items = [("add", 64, 100), ("mul", 300, 77)]
    codes, tls, want = [], [], []
    for j, (op, r, c) in enumerate(items):
        prog = _binary(op)
        a, b = wl.randn((r, c), torch.float32, 10 + j), wl.randn((r, c), torch.float32, 20 + j)
        out = torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")
        codes.append(dvm.encode(dvm.program_from_nodes(prog.nodes), [(r, c), (r, c)]))
        tls.append([a.cuda(), b.cuda(), out])
        want.append(oracle_run(prog, [a, b])[0])
    dvm.launch_stacked(codes, tls, levels=[3, 3])
    assert dvm.last_device_status() == 0
    for t, w in zip(tls, want):
        g1, _ = gate_errors(wl.to_f64(t[-1]), w)
        assert g1 <= 1e-5
