"""Seeded random programs on random views against the oracle: shapes of rank 1..4, inputs and outputs as
permuted / sliced / stepped / expanded views of larger storages, an elementwise chain with an optional
reduction over a random axis.  Every element of every output storage is compared (poison outside the view)."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc
from tests.parity_util import TORCH_DT, gate_errors

pytestmark = pytest.mark.gpu
POISON = -12288.0


def _random_view(rng, shape, allow_zero_stride):
    """A view of `shape` inside a fresh storage: dims laid out in a random order, each padded by a random
    amount, optionally stepped; some size>1 dims expanded (stride 0) when allowed.  Returns (numel, offset, strides)."""
    r = len(shape)
    order = list(rng.permutation(r))            # order[0] is the innermost dim in memory
    strides = [0] * r
    span = 1
    for k in order:
        step = int(rng.integers(1, 3)) if rng.random() < 0.3 else 1
        if allow_zero_stride and shape[k] > 1 and rng.random() < 0.15:
            strides[k] = 0
            continue
        strides[k] = span * step
        span = strides[k] * shape[k] + int(rng.integers(0, 4))
    offset = int(rng.integers(0, 6))
    return span + offset + 1, offset, strides


def _case(seed):
    rng = np.random.default_rng(seed)
    r = int(rng.integers(1, 5))
    shape = tuple(int(rng.choice([1, 2, 3, 5, 8, 17, 33, 64, 100])) for _ in range(r))
    if rng.random() < 0.3:
        shape = shape[:-1] + (int(rng.choice([257, 1000, 1531, 4096])),)
    while int(np.prod(shape)) > 400000:
        shape = shape[1:] if len(shape) > 1 else (shape[0] // 2,)
    r = len(shape)
    dt = "bf16" if rng.random() < 0.4 else "f32"
    p = wl.OpProgram(f"fuzz{seed}")
    a, b = p.input(dt, r), p.input(dt, r)
    v = p.binary(str(rng.choice(["add", "sub", "mul", "max"])), a, p.scalar("muls", b, 0.5))
    v = p.unary(str(rng.choice(["tanh", "abs", "sigmoid", "neg"])), v)
    red_axis = None
    if rng.random() < 0.5:
        red_axis = -int(rng.integers(1, r + 1))
        if shape[red_axis] > 8192:
            red_axis = None
    if red_axis is not None:
        s = p.reduce(str(rng.choice(["sum", "max", "min"])), v, red_axis)
        if rng.random() < 0.5:
            v = p.binary("sub", v, s)          # the reduced value broadcast back over its axis
        else:
            v = s
    p.output(v, dt)
    return rng, p, shape, dt, red_axis


@pytest.mark.parametrize("seed", range(160))
def test_random_program_on_random_views(seed):
    rng, p, shape, dt, red_axis = _case(seed)
    views = [_random_view(rng, shape, allow_zero_stride=True) for _ in range(2)]
    storages = [wl.randn((n,), TORCH_DT[dt], 1000 * seed + k) for k, (n, _, _) in enumerate(views)]
    hp = dvm.program_from_nodes(p.nodes)
    logical = [orc.view_load(wl.to_f64(st), off, shape, strides) for st, (_, off, strides) in zip(storages, views)]
    want = orc.evaluate(p.nodes, logical)[0]
    on, ooff, ostr = _random_view(rng, want.shape, allow_zero_stride=False)
    try:
        code = dvm.encode(hp, [shape, shape], in_strides=[v[2] for v in views], out_strides=[ostr])
    except dvm.DvmError as e:
        assert e.status == -3, e                  # a documented limit (e.g. more than three outer dims after merging)
        pytest.skip(str(e))
    assert tuple(code.out_shapes[0]) == tuple(want.shape)
    dev = [st.cuda() for st in storages]
    out = torch.full((on,), POISON, dtype=TORCH_DT[dt], device="cuda")
    es = out.element_size()
    dvm.launch(code, [d.data_ptr() + v[1] * es for d, v in zip(dev, views)] + [out.data_ptr() + ooff * es])
    assert dvm.last_device_status() == 0
    exp = orc.view_store(np.full((on,), POISON), ooff, want.shape, ostr, want)
    got = wl.to_f64(out)
    touched = exp != POISON
    assert np.array_equal(got[~touched], exp[~touched]), "an element outside the view was written"
    if want.size:
        # tolerance: row-scaled over the whole output (sums over up to 8192 elements of O(1) values)
        scale = max(1.0, float(np.max(np.abs(want))))
        tol = (2e-2 if dt == "bf16" else 1e-5) * scale * (4 if red_axis is not None else 1)
        assert float(np.max(np.abs(got[touched] - exp[touched]))) <= tol
