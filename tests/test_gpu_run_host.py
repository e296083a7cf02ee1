"""dvm_run_host: host tensors in, host tensors out (the end-to-end path bench.py times), plain and pipelined over
chunks of tiles; both against the oracle, and the pipelined result bit-equal to a plain launch's."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from oracle import dvm_oracle as orc
from tests.parity_util import gate_errors

pytestmark = pytest.mark.gpu


def _run_host(prog, ins, out_dtypes):
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [tuple(t.shape) for t in ins])
    h_in = [t.contiguous().pin_memory() for t in ins]
    h_out = [torch.full(s, float("nan"), dtype=d).pin_memory() for s, d in zip(code.out_shapes, out_dtypes)]
    total = sum(((t.numel() * t.element_size() + 255) // 256) * 256 for t in h_in + h_out)
    staging = torch.empty(total + 4096, dtype=torch.uint8, device="cuda")
    dvm.run_host(code, h_in + h_out, staging)
    assert dvm.last_device_status() == 0
    return code, h_out


@pytest.mark.parametrize("rows", [300, 5000, 20001])   # 20001 rows x 4096 bf16 x 4 tensors = 655 MB: pipelined, ragged last chunk
def test_add_rmsnorm_through_host_buffers(rows):
    prog = wl.program_add_rmsnorm(4096)
    ins = wl.inputs_add_rmsnorm(rows, 4096, seed=rows)
    code, h_out = _run_host(prog, ins, [torch.bfloat16, torch.bfloat16])
    # every row against the oracle for the small cases, blocks of rows (chunk boundaries included) for the large one
    blocks = [(0, rows)] if rows <= 5000 else [(0, 1024), (rows // 2 - 512, rows // 2 + 512), (rows - 1024, rows)]
    for r0, r1 in blocks:
        want = orc.evaluate(prog.nodes, [wl.to_f64(ins[0][r0:r1]), wl.to_f64(ins[1][r0:r1]), wl.to_f64(ins[2])])
        for g, w in zip(h_out, want):
            g1, g2 = gate_errors(wl.to_f64(g[r0:r1]), w)
            assert g2 <= 2e-2, (r0, g1, g2)
    # the same bits as one plain launch on device tensors
    dev = [t.cuda() for t in ins]
    outs = [torch.empty((rows, 4096), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    dvm.launch(code, dev + outs)
    torch.cuda.synchronize()
    for g, o in zip(h_out, outs):
        assert torch.equal(g, o.cpu())


def test_masked_softmax_through_host_buffers_takes_the_plain_way():
    """The mask is neither dense over the tiles nor a row vector: no pipelining, same result."""
    prog = wl.program_masked_softmax()
    ins = wl.inputs_masked_softmax(2, 32, 700, 5)          # 63 MB of scores + the same of output
    code, h_out = _run_host(prog, ins, [torch.bfloat16])
    want = orc.evaluate(prog.nodes, [wl.to_f64(ins[0][:1, :4]), wl.to_f64(ins[1])])[0]
    g1, g2 = gate_errors(wl.to_f64(h_out[0][:1, :4]), want)
    assert g2 <= 2e-2
    assert not torch.isnan(h_out[0].float()).any()
