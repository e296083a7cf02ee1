"""dvm_launch_stacked_noalloc: the stacked launch for callers that cannot allocate device memory.

Some users of this library run inside a memory pool that owns the whole device, or in a serving loop where
a first-use cudaMalloc (which synchronises the device) is not acceptable.  For them the library offers a
stacked launch whose work queue lives in a fixed array inside the library image.  It must give exactly what
dvm_launch_stacked gives, call after call, because every call reuses (and first clears) the same array.

This file sorts last on purpose: a run that stops at the first failure has then run every other test."""
import os
import subprocess
import sys

import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm

pytestmark = pytest.mark.gpu


def _stack(items, seed0):
    progs = {k: dvm.program_from_nodes(wl.stack_program(k).nodes) for k in wl.STACK_KINDS}
    codes, tls = [], []
    for j, (kind, r, c) in enumerate(items):
        ins, params = wl.inputs_stack(kind, r, c, seed0 + 4 * j)
        dev = [t.cuda() for t in ins]
        out = torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")
        codes.append(dvm.encode(progs[kind], [tuple(t.shape) for t in ins], params))
        tls.append(dev + [out])
    return codes, tls


def test_noalloc_matches_stacked_launch_twice_in_a_row():
    dvm.set_elems_per_thread(16)
    try:
        items = wl.shapes_c4(1)[0][:24] + [("layernorm", 1, 64), ("sigmoid_mul", 512, 4095)]
        codes, tls = _stack(items, 4242)
        dvm.launch_stacked(codes, tls)
        torch.cuda.synchronize()
        want = [t[-1].clone() for t in tls]
        assert not any(torch.isnan(w).any() for w in want)
        for call in range(2):
            for t in tls:
                t[-1].fill_(float("nan"))
            dvm.launch_stacked(codes, tls, noalloc=True)
            torch.cuda.synchronize()
            for w, t in zip(want, tls):
                # same kernel, same inputs: the tolerance of the parity tests is met with equality
                assert torch.equal(w, t[-1]), f"call {call}"
    finally:
        dvm.set_elems_per_thread(0)


_FRESH_PROCESS = r"""
import numpy as np, torch
import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc

torch.cuda.set_device(0)
dvm.set_elems_per_thread(16)
items = [("gelu_affine", 33, 300), ("layernorm", 200, 1000), ("sigmoid_mul", 64, 257), ("layernorm", 1, 64)]
progs = {k: dvm.program_from_nodes(wl.stack_program(k).nodes) for k in wl.STACK_KINDS}
codes, tls, host = [], [], []
for j, (kind, r, c) in enumerate(items):
    ins, params = wl.inputs_stack(kind, r, c, 900 + 4 * j)
    codes.append(dvm.encode(progs[kind], [tuple(t.shape) for t in ins], params))
    tls.append([t.cuda() for t in ins] + [torch.full((r, c), float("nan"), dtype=torch.float32, device="cuda")])
    host.append((kind, ins, params))

def check(tag):
    for (kind, ins, params), t in zip(host, tls):
        want = orc.evaluate(wl.stack_program(kind).nodes, [wl.to_f64(x) for x in ins], params)[0]
        got = wl.to_f64(t[-1])
        den = np.maximum(np.abs(want), np.max(np.abs(want), axis=-1, keepdims=True))
        assert np.all(np.abs(got - want) <= 1e-5 * den), (tag, kind)

assert dvm.launch_count() == 0
# the very first launch this process makes through the library: the call itself has to resolve the array's address
dvm.launch_stacked(codes, tls, noalloc=True)
torch.cuda.synchronize()
assert dvm.launch_count() == 1
check("first call")
# (the first launch of a kernel makes the driver load its code, which takes device memory whoever launches it;
#  from the second call on, free device memory must not move)
for t in tls:
    t[-1].fill_(float("nan"))
torch.cuda.synchronize()
free_before = torch.cuda.mem_get_info()[0]
dvm.launch_stacked(codes, tls, noalloc=True)
torch.cuda.synchronize()
free_after = torch.cuda.mem_get_info()[0]
check("second call")
assert free_after == free_before, (free_before, free_after)
print("NOALLOC-FRESH-OK", free_before)
"""


def test_noalloc_first_in_a_fresh_process_matches_oracle_and_takes_no_device_memory():
    """The entry point as its users meet it: the first launch a process makes through the library (so its own
    first-use set-up runs, not the regular launch's), checked against the CPU oracle, and free device memory
    identical before and after a call."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-c", _FRESH_PROCESS], cwd=root, env=env, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "NOALLOC-FRESH-OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


def test_noalloc_rejects_more_than_the_stated_maximum():
    import ctypes as C
    lib = dvm.binding.lib
    n = 257  # DVM_NOALLOC_MAX_PROGRAMS + 1
    arr = (C.c_void_p * n)()
    sz = (C.c_size_t * n)()
    tp = (C.POINTER(C.c_void_p) * n)()
    nt = (C.c_int * n)()
    assert lib.dvm_launch_stacked_noalloc(n, arr, sz, tp, nt, None) == -10
    assert lib.dvm_launch_stacked_noalloc(0, None, None, None, None, None) == 0
