"""GPU parity of stacking-based fusion: many independent programs in one launch (config 4)."""
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import record_strict, check, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[16])
def elems_per_thread(request):
    """Programs of one stacked launch share the elements-per-thread setting (16 always fits local memory)."""
    dvm.set_elems_per_thread(request.param)
    yield request.param
    dvm.set_elems_per_thread(0)


def _stack(items, seed0):
    progs = {k: wl.stack_program(k) for k in wl.STACK_KINDS}
    ps = {k: dvm.program_from_nodes(p.nodes) for k, p in progs.items()}
    codes, tls, meta = [], [], []
    for j, (kind, r, c) in enumerate(items):
        ins, params = wl.inputs_stack(kind, r, c, seed0 + 4 * j)
        dev = [t.cuda() for t in ins]
        out = torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")
        codes.append(dvm.encode(ps[kind], [tuple(t.shape) for t in ins], params))
        tls.append(dev + [out])
        meta.append((progs[kind], ins, params, out, kind))
    return codes, tls, meta


def _check_all(meta, report=None):
    for j, (prog, ins, params, out, kind) in enumerate(meta):
        want = oracle_run(prog, ins, params)
        check(prog, [out], want, strict=(kind == "sigmoid_mul"))
        if report and kind != "sigmoid_mul":
            st = record_strict(f"{report} #{j} {kind} {tuple(out.shape)}", prog, [out], ins, params, want_list=want)[0]
            # elements a faithful fp32 evaluation gets right must not be lost by the device (the row-scaled gate
            # alone would not notice a small output that was zeroed)
            assert st["well_max"] <= 5e-2, st


def test_stacked_small_mix():
    items = [("gelu_affine", 3, 65), ("layernorm", 17, 100), ("sigmoid_mul", 1, 64), ("layernorm", 1, 4096),
             ("gelu_affine", 200, 333), ("sigmoid_mul", 511, 4095), ("layernorm", 512, 64)]
    codes, tls, meta = _stack(items, 100)
    dvm.launch_stacked(codes, tls)
    assert dvm.last_device_status() == 0
    _check_all(meta)


@pytest.mark.parametrize("min_ctas,launch", [(0, 0), (2, 0), (2, 1), (2, 7)])
def test_stacked_config4_launches(min_ctas, launch):
    """Seeded launches of config 4: 64 programs, one kernel; with dvm_set_min_resident_ctas(2) in the
    configuration bench.py times (geometries costed by total work, two CTAs per SM)."""
    items = wl.shapes_c4(launch + 1)[launch]
    assert len(items) == 64
    dvm.set_min_resident_ctas(min_ctas)
    try:
        codes, tls, meta = _stack(items, wl.data_seed("c4", 0) + launch)
    finally:
        dvm.set_min_resident_ctas(0)
    n0 = dvm.launch_count()
    dvm.launch_stacked(codes, tls)
    assert dvm.last_device_status() == 0
    assert dvm.launch_count() - n0 == 1
    _check_all(meta, report=f"c4 launch {launch}" if (min_ctas, launch) == (2, 0) else None)


@pytest.mark.parametrize("launch", [0, 3])
def test_stacked_config4_launches_one_slot_per_cta(launch):
    """The configuration bench.py times for config 4: 32 elements per thread, geometries that fit two CTAs with
    one tile slot each (dvm_set_min_resident_ctas(3)), launched with dvm_set_stacked_one_slot."""
    items = wl.shapes_c4(launch + 1)[launch]
    dvm.set_elems_per_thread(32)
    dvm.set_min_resident_ctas(3)
    dvm.set_stacked_one_slot(True)
    try:
        codes, tls, meta = _stack(items, wl.data_seed("c4", 0) + launch)
        n0 = dvm.launch_count()
        dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
        assert dvm.launch_count() - n0 == 1
        # a second launch of the same programs finds the queue counters at rest
        for t in tls:
            t[-1].fill_(float("nan"))
        dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
    finally:
        dvm.set_min_resident_ctas(0)
        dvm.set_stacked_one_slot(False)
    _check_all(meta)


def test_stacked_repeated_launches_reuse_queue():
    """The work queue returns to its resting state after every launch."""
    items = wl.shapes_c4(2)[1][:16]
    codes, tls, meta = _stack(items, 999)
    for _ in range(5):
        for t in tls:
            t[-1].fill_(float("nan"))
        dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
        _check_all(meta)


def test_stacked_with_32_elements_per_thread():
    dvm.set_elems_per_thread(32)
    items = [("layernorm", 17, 100), ("sigmoid_mul", 300, 5000), ("layernorm", 64, 8000), ("sigmoid_mul", 200, 1024)]
    codes, tls, meta = _stack(items, 77)
    dvm.launch_stacked(codes, tls)
    assert dvm.last_device_status() == 0
    _check_all(meta)


def test_stacked_rejects_mixed_settings():
    dvm.set_elems_per_thread(16)
    c1, t1, _ = _stack([("sigmoid_mul", 5, 70)], 5)
    dvm.set_elems_per_thread(32)
    c2, t2, _ = _stack([("sigmoid_mul", 5, 70)], 6)
    with pytest.raises(dvm.DvmError) as e:
        dvm.launch_stacked(c1 + c2, t1 + t2)
    assert e.value.status == -1


def test_stacked_one_and_empty():
    codes, tls, meta = _stack([("sigmoid_mul", 5, 70)], 5)
    dvm.launch_stacked(codes, tls)
    assert dvm.last_device_status() == 0
    _check_all(meta)
    dvm.launch_stacked([], [])


def test_stacked_equals_separate_launches():
    items = wl.shapes_c4(3)[2][:12]
    codes, tls, meta = _stack(items, 31337)
    dvm.launch_stacked(codes, tls)
    torch.cuda.synchronize()
    stacked = [t[-1].clone() for t in tls]
    for c, t in zip(codes, tls):
        t[-1].fill_(float("nan"))
        dvm.launch(c, t)
    torch.cuda.synchronize()
    for a, t in zip(stacked, tls):
        assert torch.equal(a, t[-1])


@pytest.mark.parametrize("v", [16, 32])
def test_stacked_with_two_resident_ctas_per_sm(v):
    """dvm_set_min_resident_ctas(2): every program's tile slots fit twice per SM; wide rows with row-vector
    operands then run in two or more column blocks, whose slice of the row vector is loaded with every tile."""
    dvm.set_elems_per_thread(v)
    dvm.set_min_resident_ctas(2)
    try:
        items = [("gelu_affine", 337, 3249), ("gelu_affine", 148, 2893), ("gelu_affine", 5, 4096), ("layernorm", 64, 4096),
                 ("sigmoid_mul", 511, 4095), ("gelu_affine", 40, 2049), ("gelu_affine", 3, 65), ("layernorm", 17, 100)]
        codes, tls, meta = _stack(items, 321)
        for c in codes:
            words = torch.frombuffer(bytearray(c.bytes()), dtype=torch.int32)
            units = (int(words[19]) >> 16) & 0xffff          # local-memory units of one tile slot
            assert units <= 225 or v == 32                   # (at 32 elements per thread not every program can)
        dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
        _check_all(meta)
        for c, t in zip(codes, tls):                         # and each program on its own
            t[-1].fill_(float("nan"))
            dvm.launch(c, t)
        assert dvm.last_device_status() == 0
        _check_all(meta)
    finally:
        dvm.set_min_resident_ctas(0)
