"""Random shapes with every input and output starting a random number of elements into a 16-byte word: the four
single-program sweeps' programs (if-else-add fp32, add + RMSNorm, masked softmax, the head-transpose view) against
the oracle, on whichever interpreter build the launch picks -- small instances (one tile per CTA) and instances of
hundreds to thousands of tiles (several tiles per CTA, both tile slots, wrap-around rows on the general interpreter).
Storage around every output must stay untouched."""
import collections

import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import TORCH_DT, check, oracle_run

pytestmark = pytest.mark.gpu


def _shifted(shape, dtype, seed, sh):
    n = int(np.prod(shape))
    base = wl.randn((n + 16,), dtype, seed).cuda()
    return base[sh:sh + n].view(*shape)


def _guarded_out(shape, dtype, sh):
    n = int(np.prod(shape))
    base = torch.full((n + 16,), float("nan"), dtype=dtype, device="cuda")
    return base, base[sh:sh + n].view(*shape)


def _launch_and_check(prog, code, ins, outs, bases, shifts, want, seen):
    dvm.launch(code, ins + outs)
    assert dvm.last_device_status() == 0
    v = dvm.last_launch_variant()
    seen[(v["lean"], v["ctas"], v["V"])] += 1
    check(prog, outs, want)
    for base, out, sh in zip(bases, outs, shifts):
        assert torch.isnan(base[:sh]).all() and torch.isnan(base[sh + out.numel():]).all()


@pytest.mark.parametrize("seed,n_cases,big", [(1, 120, False), (2, 40, True)])
def test_random_alignments_of_every_operand(seed, n_cases, big):
    rng = np.random.default_rng(seed)
    seen = collections.Counter()
    for it in range(n_cases):
        kind = int(rng.integers(0, 4))
        aligned = rng.random() < 0.4     # a fair share of fully aligned cases

        def sh():
            return 0 if aligned else int(rng.integers(0, 8))
        s0 = 1000 + 10 * it
        if kind == 0:
            shape = (int(rng.integers(1, 6)) * (8 if big else 1), int(rng.integers(1, 40)) * (8 if big else 1),
                     int(rng.choice([8, 64, 1000, 1001, 1024, 4099, int(rng.integers(1, 3000))])))
            prog = wl.program_if_else_add()
            ins = [_shifted(shape, torch.float32, s0 + i, sh()) for i in range(4)]
        elif kind == 1:
            cols = int(rng.choice([4096, 4000, 4001, 2048, 1536, 1000, 264]))
            rows = int(rng.integers(1, 70)) * (40 if big else 1)
            prog = wl.program_add_rmsnorm(cols)
            ins = [_shifted((rows, cols), torch.bfloat16, s0, sh()), _shifted((rows, cols), torch.bfloat16, s0 + 1, sh()),
                   _shifted((cols,), torch.bfloat16, s0 + 2, sh())]
        elif kind == 2:
            S = int(rng.choice([256, 248, 250, 128, 512, 509, 384, int(rng.integers(17, 600))] + ([1024, 2048, 1236] if big else [])))
            B, H = int(rng.integers(1, 3)), int(rng.integers(1, 5))
            prog = wl.program_masked_softmax(128)
            ins = [_shifted((B, H, S, S), torch.bfloat16, s0, sh()), wl.causal_mask(S, "cuda")]
        else:
            B, S, H, D = int(rng.integers(1, 3)), int(rng.integers(1, 300)) * (4 if big else 1), 32, 128
            prog = wl.program_head_transpose_add()
            n, shp = B * S * H * D, (B, H, S, D)
            xs, y = _shifted((n,), torch.bfloat16, s0, sh()), _shifted((n,), torch.bfloat16, s0 + 1, sh())
            code = dvm.encode(dvm.program_from_nodes(prog.nodes), [shp, shp], in_strides=[[S * H * D, D, H * D, 1], None])
            so = sh()
            base, out = _guarded_out((n,), torch.bfloat16, so)
            want = oracle_run(prog, [xs.view(B, S, H, D).permute(0, 2, 1, 3).contiguous().cpu(), y.view(shp).cpu()])
            try:
                _launch_and_check(prog, code, [xs, y], [out], [base], [so], [w.reshape(-1) for w in want], seen)
            except AssertionError as e:
                raise AssertionError(f"case {it}: views {shp}: {e}") from e
            continue
        code = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins])
        shifts = [sh() for _ in prog.output_nodes]
        pairs = [_guarded_out(shp, TORCH_DT[node[2]], s) for shp, node, s in zip(code.out_shapes, prog.output_nodes, shifts)]
        want = oracle_run(prog, [t.cpu() for t in ins])
        try:
            _launch_and_check(prog, code, ins, [o for _, o in pairs], [b for b, _ in pairs], shifts, want, seen)
        except AssertionError as e:
            raise AssertionError(f"case {it}: {prog.name} {[tuple(t.shape) for t in ins]}: {e}") from e
    # the sweep reached the lean builds and the general interpreter, on two and on three CTAs per SM
    leans = {k[0] for k in seen}
    assert {0, 1, 3, 4, 9} <= leans and any(k[1] == 3 for k in seen), dict(seen)


def _guards_ok(base, out, sh):
    if base.dtype.is_floating_point:
        return bool(torch.isnan(base[:sh]).all() and torch.isnan(base[sh + out.numel():]).all())
    return bool((base[:sh] == 123).all() and (base[sh + out.numel():] == 123).all())


@pytest.mark.parametrize("seed,n_launches,big", [(1, 60, False), (2, 15, True)])
def test_random_alignments_in_stacked_launches(seed, n_launches, big):
    """Stacked launches of one to eight fp32 programs of the config-4 mix, every tensor at a random element offset, in
    the three encodings a stacked launch runs with (two slots; two resident CTAs; one slot on three CTAs per SM)."""
    rng = np.random.default_rng(seed)
    seen = collections.Counter()
    for it in range(n_launches):
        mode = int(rng.integers(0, 3))
        aligned = rng.random() < 0.3

        def sh():
            return 0 if aligned else int(rng.integers(0, 4))
        dvm.set_elems_per_thread(32 if rng.random() < 0.7 else 16)   # (the programs of a launch share one tile shape)
        if mode == 1:
            dvm.set_min_resident_ctas(2)
        if mode == 2:
            dvm.set_min_resident_ctas(3)
            dvm.set_stacked_one_slot(True)
        try:
            progs, codes, tls, outs = [], [], [], []
            for k in range(int(rng.integers(1, 9))):
                kind = int(rng.integers(0, 3))
                rows = int(rng.integers(1, 400)) * (6 if big else 1)
                cols = int(rng.choice([27, 320, 1000, 1001, 1024, 2048, 2173, 4096, int(rng.integers(1, 5000))]))
                s0, params = 5000 + 100 * it + 10 * k, ()
                if kind == 0:
                    prog = wl.program_gelu_affine()
                    ins = [_shifted((rows, cols), torch.float32, s0, sh()), _shifted((1, cols), torch.float32, s0 + 1, sh()),
                           _shifted((1, cols), torch.float32, s0 + 2, sh())]
                elif kind == 1:
                    prog, params = wl.program_layernorm(), (1.0 / cols,)
                    ins = [_shifted((rows, cols), torch.float32, s0, sh())]
                else:
                    prog = wl.program_sigmoid_mul()
                    ins = [_shifted((rows, cols), torch.float32, s0, sh()), _shifted((rows, cols), torch.float32, s0 + 1, sh())]
                try:
                    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins], params)
                except dvm.DvmError:
                    continue   # (a row longer than this encoding's tile)
                so = sh()
                base, out = _guarded_out((rows, cols), torch.float32, so)
                progs.append((prog, params, ins)); codes.append(code); tls.append(ins + [out]); outs.append((base, out, so))
            if not codes:
                continue
            dvm.launch_stacked(codes, tls)
            assert dvm.last_device_status() == 0
            v = dvm.last_launch_variant()
            seen[(mode, v["ctas"], v["V"])] += 1
            for (prog, params, ins), (base, out, so) in zip(progs, outs):
                check(prog, [out], oracle_run(prog, [t.cpu() for t in ins], params))
                assert _guards_ok(base, out, so), (it, prog.name)
        finally:
            dvm.set_min_resident_ctas(0)
            dvm.set_stacked_one_slot(False)
            dvm.set_elems_per_thread(0)
    assert any(k[1] == 3 for k in seen) and any(k[1] == 2 for k in seen), dict(seen)


def test_random_alignments_of_long_rows_and_integer_outputs():
    """Rows longer than a tile (programs in phases) and integer outputs (a u8 mask, i32 / u8 casts; offsets of 1 to
    15 elements, so byte stores at every phase of a 16-byte word), every tensor at a random element offset."""
    from tests.test_gpu_int_types import _safe_inputs
    rng = np.random.default_rng(3)
    for it in range(70):
        kind = int(rng.integers(0, 5))
        aligned = rng.random() < 0.3

        def sh(lim=8):
            return 0 if aligned else int(rng.integers(0, lim))
        s0, params = 9000 + 10 * it, ()
        if kind <= 1:       # long rows
            rows = int(rng.integers(1, 300))
            cols = int(rng.choice([8200, 8192, 12345, 16384, 20000, int(rng.integers(4097, 40000))]))
            if kind == 0:
                prog, params = wl.program_layernorm(), (1.0 / cols,)
                ins = [_shifted((rows, cols), torch.float32, s0, sh())]
            else:
                prog = wl.program_add_rmsnorm(cols)
                ins = [_shifted((rows, cols), torch.bfloat16, s0, sh()), _shifted((rows, cols), torch.bfloat16, s0 + 1, sh()),
                       _shifted((cols,), torch.bfloat16, s0 + 2, sh())]
        elif kind == 2:
            shape = (int(rng.integers(1, 5)), int(rng.integers(1, 40)), int(rng.choice([8, 333, 1000, 4096, 4099, int(rng.integers(1, 3000))])))
            prog = wl.program_if_else_add_mask()
            ins = [_shifted(shape, torch.float32, s0 + i, sh()) for i in range(4)]
        else:
            shape = (int(rng.integers(1, 300)), int(rng.choice([63, 1000, 1531, 4096, 4000, int(rng.integers(1, 4500))])))
            in_dtype = "f32" if kind == 3 else "bf16"
            prog = wl.program_quantise(in_dtype)
            x = _safe_inputs(shape, torch.bfloat16 if in_dtype == "bf16" else torch.float32, it + 3, 10.0)
            holder = torch.empty((x.numel() + 16,), dtype=x.dtype, device="cuda")
            s = sh()
            holder[s:s + x.numel()] = x.reshape(-1).cuda()
            ins = [holder[s:s + x.numel()].view(*shape)]
        code = dvm.encode(dvm.program_from_nodes(prog.nodes), [tuple(t.shape) for t in ins], params)
        outs = []
        for shp, node in zip(code.out_shapes, prog.output_nodes):
            dt, so, n = TORCH_DT[node[2]], sh(16), int(np.prod(shp))
            base = torch.full((n + 16,), float("nan") if dt.is_floating_point else 123, dtype=dt, device="cuda")
            outs.append((base, base[so:so + n].view(*shp), so))
        dvm.launch(code, ins + [o for _, o, _ in outs])
        assert dvm.last_device_status() == 0
        want = oracle_run(prog, [t.cpu() for t in ins], params)
        for (base, out, so), w, node in zip(outs, want, prog.output_nodes):
            if node[2] in ("u8", "i32"):
                assert np.array_equal(out.cpu().numpy().astype(np.float64), w), (it, prog.name, node[2])
            else:
                check(prog, [out], [w])
            assert _guards_ok(base, out, so), (it, prog.name)


def test_random_alignments_of_matmul_epilogue_operands():
    """addmm (Table 2) with its epilogue operand -- [m,n], [1,n] or [m,1] -- and its output at random element offsets
    (the matrices A and B stay 16-byte aligned: the tile loads need that, and the launch refuses anything else)."""
    from tests.parity_util import gate_errors
    rng = np.random.default_rng(4)
    prog = wl.program_addmm()
    for it in range(50):
        M = int(rng.choice([1, 7, 100, 128, 129, 300, 1000, int(rng.integers(1, 1500))]))
        K, N = int(rng.choice([64, 256, 512, 1024])), int(rng.choice([64, 256, 264, 512, 1000, 1024]))
        cshape = [(M, N), (1, N), (M, 1)][int(rng.integers(0, 3))]
        sc, so = int(rng.integers(0, 8)), int(rng.integers(0, 8))
        a = (wl.randn((M, K), torch.bfloat16, 100 + it) * 0.25).cuda()
        b = (wl.randn((K, N), torch.bfloat16, 200 + it) * 0.25).cuda()
        c = _shifted(cshape, torch.bfloat16, 300 + it, sc)
        base, out = _guarded_out((M, N), torch.bfloat16, so)
        code = dvm.encode(dvm.program_from_nodes(prog.nodes), [(M, K), (K, N), cshape])
        dvm.launch(code, [a, b, c, out])
        assert dvm.last_device_status() == 0
        g1, _ = gate_errors(wl.to_f64(out), oracle_run(prog, [a.cpu(), b.cpu(), c.cpu()])[0])
        assert g1 <= 2e-2, (it, M, K, N, cshape, sc, so, g1)
        assert _guards_ok(base, out, so), (it, M, K, N, cshape, sc, so)
    a = wl.randn((128 * 64 + 8,), torch.bfloat16, 1).cuda()[1:1 + 128 * 64].view(128, 64)   # A two bytes off: refused
    with pytest.raises(dvm.DvmError):
        dvm.launch(dvm.encode(dvm.program_from_nodes(wl.program_matmul().nodes), [(128, 64), (64, 64)]),
                   [a, torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda"), torch.empty((128, 64), dtype=torch.bfloat16, device="cuda")])
