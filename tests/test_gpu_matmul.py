"""GPU parity of the matmul meta-kernel (tcgen05 matmul instruction + interpreted epilogue) against the
CPU oracle: every output element at small sizes (ragged M, N and K tails, several tiles), sampled rows at
the full size of config 5, special cases with exact answers, and epilogues with extra operands."""
import numpy as np
import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gate_errors, gpu_run, oracle_run, record_strict

pytestmark = pytest.mark.gpu

R_BF16 = 2e-2  # bf16 programs, fp32 accumulation


def _mlp_inputs(M, K, N, seed):
    x = wl.randn((M, K), torch.bfloat16, seed)
    wg = wl.randn((K, N), torch.bfloat16, seed + 1, std=0.02)
    wu = wl.randn((K, N), torch.bfloat16, seed + 2, std=0.02)
    return [x, wg, wu]


@pytest.mark.parametrize("M,K,N", [(1, 64, 128), (7, 64, 128), (128, 64, 128), (129, 128, 256), (77, 200, 264),
                                   (300, 1024, 392), (257, 4096, 512), (128, 72, 8), (5, 8, 8)])
def test_mlp_gate_small(M, K, N):
    """out = SiLU(X Wg) * (X Wu): every element, row-scaled gate at 2e-2."""
    ins = _mlp_inputs(M, K, N, seed=M + N)
    outs, code = gpu_run(wl.program_mlp_gate(), ins)
    want = oracle_run(wl.program_mlp_gate(), ins)
    g1, _ = check(wl.program_mlp_gate(), outs, want)
    assert not torch.isnan(outs[0].float()).any()  # every element of the poisoned output was written


def test_mlp_gate_config_shape_rows():
    """Config 5 geometry (K = 4096, N = 11008) at a token count the oracle finishes in seconds."""
    M, K, N = 200, 4096, 11008
    w = wl.mlp_weights(K, N)
    ins = wl.inputs_mlp_gate(M, K, N, seed=wl.data_seed("c5", 0), weights=w)
    outs, _ = gpu_run(wl.program_mlp_gate(), ins)
    want = oracle_run(wl.program_mlp_gate(), ins)
    check(wl.program_mlp_gate(), outs, want)
    st = record_strict("c5 SiLU(X Wg) * (X Wu) M=200", wl.program_mlp_gate(), outs, ins, want_list=want)[0]
    # outputs that fp32 accumulation gets right are right on the device too, up to the bf16 rounding of the store
    assert st["n_well"] > 0.5 * st["n"] and st["well_max"] <= 8e-3, st


def test_mlp_gate_full_size_sampled_rows():
    """M = 4096 (the largest instance of config 5, the launch the bench times): 48 sampled rows, one by one."""
    M, K, N = 4096, 4096, 11008
    w = wl.mlp_weights(K, N)
    ins = wl.inputs_mlp_gate(M, K, N, seed=wl.data_seed("c5", 1), weights=w)
    outs, _ = gpu_run(wl.program_mlp_gate(), ins)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 127, 128, 4095], rng.integers(0, M, 44)]))
    sub = [ins[0][rows], ins[1], ins[2]]
    want = oracle_run(wl.program_mlp_gate(), sub)
    got = wl.to_f64(outs[0])[rows]
    g1, _ = gate_errors(got, want[0])
    assert g1 <= R_BF16, g1
    assert not torch.isnan(outs[0].float()).any()


def _plain_matmul(out_dtype="bf16"):
    p = wl.OpProgram("matmul")
    a, b = p.input("bf16", 2), p.input("bf16", 2)
    p.output(p.matmul(a, b), out_dtype)
    return p


@pytest.mark.parametrize("M,K,N", [(64, 64, 256), (130, 136, 520), (1, 4096, 264)])
def test_plain_matmul_f32_out(M, K, N):
    """One B matrix (256-column tiles), fp32 output: products of bf16 are exact in fp32, so only the
    accumulation order differs from the oracle: 1e-5 row-scaled."""
    a = wl.randn((M, K), torch.bfloat16, 11)
    b = wl.randn((K, N), torch.bfloat16, 12)
    prog = _plain_matmul("f32")
    outs, _ = gpu_run(prog, [a, b])
    want = oracle_run(prog, [a, b])
    g1, _ = gate_errors(wl.to_f64(outs[0]), want[0])
    assert g1 <= 1e-5, g1


def test_identity_picks_out_b():
    """X = I (K = 128) returns B exactly, element by element (each product has a single non-zero term)."""
    K, N = 128, 384
    b = wl.randn((K, N), torch.bfloat16, 3)
    a = torch.eye(K, dtype=torch.bfloat16)
    outs, _ = gpu_run(_plain_matmul("bf16"), [a, b])
    assert torch.equal(outs[0].cpu(), b)


def test_permutation_rows():
    """A row permutation matrix as X permutes the rows of B exactly (catches a transposed or swizzled operand)."""
    K, N = 192, 264
    perm = torch.randperm(K, generator=torch.Generator().manual_seed(4))
    a = torch.zeros((K, K), dtype=torch.bfloat16)
    a[torch.arange(K), perm] = 1
    b = wl.randn((K, N), torch.bfloat16, 5)
    outs, _ = gpu_run(_plain_matmul("bf16"), [a, b])
    assert torch.equal(outs[0].cpu(), b[perm])


def test_zero_gate_gives_zero():
    M, K, N = 100, 256, 256
    x = wl.randn((M, K), torch.bfloat16, 1)
    wu = wl.randn((K, N), torch.bfloat16, 2)
    outs, _ = gpu_run(wl.program_mlp_gate(), [x, torch.zeros((K, N), dtype=torch.bfloat16), wu])
    assert torch.all(outs[0] == 0)


def test_all_ones_closed_form():
    """All-ones operands: g = u = K, out = K * sigmoid(K) * K."""
    M, K, N = 130, 64, 136
    one = lambda *s: torch.ones(s, dtype=torch.bfloat16)
    outs, _ = gpu_run(wl.program_mlp_gate(), [one(M, K), one(K, N), one(K, N)])
    want = torch.tensor(K * K / (1 + np.exp(-K)), dtype=torch.float64).to(torch.bfloat16)
    assert torch.all(outs[0].cpu() == want)


def test_epilogue_with_extra_operands_and_temporaries():
    """addmm-like epilogue: bias row vector, residual matrix, a column vector, two outputs, a spilled value."""
    M, K, N = 150, 192, 392
    p = wl.OpProgram("addmm_chain")
    x, w = p.input("bf16", 2), p.input("bf16", 2)
    bias, res, colv = p.input("f32", 1), p.input("bf16", 2), p.input("f32", 2)
    g = p.matmul(x, w)
    t = p.binary("add", g, bias)
    u = p.binary("sub", res, p.unary("tanh", t))
    v = p.binary("mul", p.binary("mul", u, t), colv)
    p.output(p.scalar("muls", v, 0.5), "f32")
    p.output(t, "bf16")
    ins = [wl.randn((M, K), torch.bfloat16, 1), wl.randn((K, N), torch.bfloat16, 2, std=0.05),
           wl.randn((N,), torch.float32, 3), wl.randn((M, N), torch.bfloat16, 4), wl.randn((M, 1), torch.float32, 5)]
    outs, code = gpu_run(p, ins)
    want = oracle_run(p, ins)
    check(p, outs, want)


def test_two_launches_same_code_other_buffers():
    """Bytecode holds tensor slots, not addresses: one encoded program runs on other buffers."""
    M, K, N = 140, 128, 256
    prog = wl.program_mlp_gate()
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [(M, K), (K, N), (K, N)])
    for seed in (1, 2):
        ins = _mlp_inputs(M, K, N, seed)
        dev = [t.cuda() for t in ins]
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        dvm.launch(code, dev + [out])
        assert dvm.last_device_status() == 0
        check(prog, [out], oracle_run(prog, ins))


def test_empty_m_launches_nothing():
    prog = wl.program_mlp_gate()
    p = dvm.program_from_nodes(prog.nodes)
    code = dvm.encode(p, [(0, 64), (64, 128), (64, 128)])
    x = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((0, 128), dtype=torch.bfloat16, device="cuda")
    n0 = dvm.launch_count()
    dvm.launch(code, [x, w, w.clone(), out])
    assert dvm.launch_count() == n0


@pytest.mark.parametrize("m,n,k", [(1, 4096, 4096), (200, 11008, 4096), (130, 4096, 11008), (257, 5120, 5120),
                                   (77, 13696, 5120), (300, 5120, 13696), (129, 8192, 8192)])
def test_addmm_llm_shapes_small_m(m, n, k):
    """addmm = matmul + fused add of a [m,n] operand (Table 2 shapes at token counts the oracle finishes in
    seconds): every element."""
    prog = wl.program_addmm()
    ins = [wl.randn((m, k), torch.bfloat16, m), wl.randn((k, n), torch.bfloat16, n, std=0.02),
           wl.randn((m, n), torch.bfloat16, k)]
    outs, _ = gpu_run(prog, ins)
    check(prog, outs, oracle_run(prog, ins))
    assert not torch.isnan(outs[0].float()).any()


@pytest.mark.parametrize("m,n,k", [(8192, 28672, 8192), (6000, 8192, 28672)])
def test_addmm_largest_shapes_sampled_rows(m, n, k):
    """The largest (n, k) pairs of Table 2 at large m: sampled rows against the oracle, one by one."""
    prog = wl.program_addmm()
    a = wl.randn((m, k), torch.bfloat16, 1, "cuda")
    b = wl.randn((k, n), torch.bfloat16, 2, "cuda", std=0.02)
    c = wl.randn((m, n), torch.bfloat16, 3, "cuda")
    out = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device="cuda")
    code = dvm.encode(dvm.program_from_nodes(prog.nodes), [(m, k), (k, n), (m, n)])
    dvm.launch(code, [a, b, c, out])
    assert dvm.last_device_status() == 0
    rows = np.unique(np.concatenate([[0, 127, 128, m - 1], np.random.default_rng(7).integers(0, m, 12)]))
    ti = torch.from_numpy(rows).cuda()
    want = oracle_run(prog, [a[ti].cpu(), b.cpu(), c[ti].cpu()])
    g1, _ = gate_errors(wl.to_f64(out[ti]), want[0])
    assert g1 <= R_BF16, g1
    assert not torch.isnan(out.float().sum())


# ---- tail split: the tiles of the last, partial wave computed by several CTAs, a share of the k blocks each ----

def _tail_case(kind, M, K, N, seed):
    if kind == "mlp":
        return wl.program_mlp_gate(), _mlp_inputs(M, K, N, seed)
    a = wl.randn((M, K), torch.bfloat16, seed)
    b = wl.randn((K, N), torch.bfloat16, seed + 1, std=0.02)
    c = wl.randn((M, N), torch.bfloat16, seed + 2)
    return wl.program_addmm(), [a, b, c]


@pytest.mark.parametrize("kind,M,K,N", [
    ("addmm", 128, 1088, 2560),    # one wave of 10 tiles: four CTAs per tile, 17 k blocks shared 5 / 5 / 5 / 2
    ("addmm", 1024, 1024, 4864),   # 152 tiles: a full wave, then 4 tiles by four CTAs each
    ("mlp", 256, 1024, 12672),     # 198 tiles of both products: a full wave, then 50 tiles by two CTAs each
    ("mlp", 100, 2048, 3200),      # one wave of 25 tiles, ragged M: four CTAs per tile (the cap)
    ("addmm", 77, 1600, 9000),     # ragged M, N and a k tail: 36 tiles, four CTAs each
])
def test_tail_split_against_oracle_and_unsplit(kind, M, K, N):
    prog, ins = _tail_case(kind, M, K, N, seed=M + N + K)
    try:
        dvm.set_matmul_tail_split(True)
        outs, _ = gpu_run(prog, ins)
        again, _ = gpu_run(prog, ins)
        dvm.set_matmul_tail_split(False)
        plain, _ = gpu_run(prog, ins)
    finally:
        dvm.set_matmul_tail_split(True)
    want = oracle_run(prog, ins)
    check(prog, outs, want)
    check(prog, plain, want)
    assert not torch.isnan(outs[0].float()).any()
    # the shares are added in a fixed order: the same bits every time
    assert torch.equal(outs[0], again[0])
    # against the unsplit accumulation only the fp32 rounding of the partial sums differs: a bf16 step at most
    a, b = outs[0].float(), plain[0].float()
    scale = b.abs().max().item()
    assert (a - b).abs().max().item() <= 2.0 ** -7 * scale
    assert (a != b).float().mean().item() < 0.2


def test_tail_split_on_two_streams():
    """Every stream has a workspace of its own: launches of two streams may overlap."""
    prog, ins = _tail_case("addmm", 128, 2048, 2560, seed=9)
    want = oracle_run(prog, ins)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    res = []
    for _ in range(3):
        for s in (s1, s2):
            res.append(gpu_run(prog, ins, stream=s)[0])
    torch.cuda.synchronize()
    for outs in res:
        check(prog, outs, want)
        assert torch.equal(outs[0], res[0][0])


# ---- CTA pairs: two CTAs of a cluster on one tile of 256 rows (tcgen05 cta_group::2) ----

@pytest.mark.parametrize("kind,M,K,N", [
    ("addmm", 256, 128, 256),      # one tile of a pair
    ("addmm", 129, 200, 264),      # the second CTA's rows end after one; ragged k and n
    ("mlp", 300, 512, 392),        # three blocks of 128 rows: the last pair's second half is empty
    ("mlp", 1024, 4096, 1536),     # both products side by side in the accumulators, 64 k blocks through 6 stages
    ("addmm", 1000, 2048, 5000),   # 80 tiles of 256 rows: more than the device runs pairs at a time
])
def test_cta_pairs_equal_single_cta_kernel(kind, M, K, N):
    prog, ins = _tail_case(kind, M, K, N, seed=M + K)
    try:
        dvm.set_matmul_tail_split(False)
        dvm.set_matmul_cta_pairs(0)
        single, _ = gpu_run(prog, ins)
        dvm.set_matmul_cta_pairs(2)
        pairs, _ = gpu_run(prog, ins)
    finally:
        dvm.set_matmul_tail_split(True)
        dvm.set_matmul_cta_pairs(1)
    check(prog, pairs, oracle_run(prog, ins))
    assert not torch.isnan(pairs[0].float()).any()
    assert torch.equal(pairs[0], single[0])  # the same k order, the same instruction shape along k


def test_cta_pairs_default_choice_keeps_parity():
    """The default mode picks pairs or single CTAs per launch; both routes against the oracle at one shape each."""
    for M, K, N in ((2048, 1024, 4096), (128, 1024, 4096)):
        prog, ins = _tail_case("addmm", M, K, N, seed=3)
        outs, _ = gpu_run(prog, ins)
        check(prog, outs, oracle_run(prog, ins))


@pytest.mark.parametrize("kind,M,K,N", [
    ("addmm", 256, 1024, 512),     # two tiles of 256 rows: four pairs each, 16 k blocks shared 4 / 4 / 4 / 4
    ("mlp", 512, 2048, 1280),      # 20 tiles: three pairs each
    ("addmm", 4096, 1088, 4864),   # 304 tiles: four full waves of pairs, then 8 tiles by four pairs each, 17 k blocks
    ("mlp", 300, 1024, 3000),      # the last pair's second CTA holds 44 rows; ragged n
])
def test_tail_split_on_cta_pairs(kind, M, K, N):
    prog, ins = _tail_case(kind, M, K, N, seed=M + N)
    try:
        dvm.set_matmul_cta_pairs(2)
        outs, _ = gpu_run(prog, ins)
        again, _ = gpu_run(prog, ins)
        dvm.set_matmul_tail_split(False)
        plain, _ = gpu_run(prog, ins)
    finally:
        dvm.set_matmul_tail_split(True)
        dvm.set_matmul_cta_pairs(1)
    want = oracle_run(prog, ins)
    check(prog, outs, want)
    check(prog, plain, want)
    assert not torch.isnan(outs[0].float()).any()
    assert torch.equal(outs[0], again[0])
    a, b = outs[0].float(), plain[0].float()
    assert (a - b).abs().max().item() <= 2.0 ** -7 * b.abs().max().item()


def test_matmul_launch_inside_a_cuda_graph():
    """A captured matmul launch replays correctly on new data: launches into a capturing stream never use the
    tail split (a replay would meet the flags of its own earlier run), pairs and single CTAs both replay."""
    for M, K, N in ((128, 1024, 2560), (1024, 1024, 4864)):   # shapes that split when launched directly
        prog, ins = _tail_case("addmm", M, K, N, seed=21)
        p = dvm.program_from_nodes(prog.nodes)
        dev = [t.cuda() for t in ins]
        code = dvm.encode(p, [tuple(t.shape) for t in dev])
        out = torch.empty(code.out_shapes[0], dtype=torch.bfloat16, device="cuda")
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            dvm.launch(code, dev + [out], s)   # set-up outside the capture
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            dvm.launch(code, dev + [out], s)
        for rep in range(3):
            dev[0].copy_(wl.randn((M, K), torch.bfloat16, 100 + rep).cuda())
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            assert dvm.last_device_status() == 0
            want = oracle_run(prog, [dev[0].cpu(), ins[1], ins[2]])
            check(prog, [out], want)


@pytest.mark.parametrize("pairs,kind,M,K,N", [
    (0, "addmm", 128, 16384, 20480),   # one wave of 80 tiles on 148 CTAs: ranges of 139 of the 256 k blocks, tiles in two or three parts
    (0, "addmm", 1024, 16384, 7424),   # 232 tiles: a full wave, then 84 tiles in ranges of 146 k blocks
    (2, "addmm", 256, 16384, 10240),   # 40 tiles of 256 rows on 74 pairs: ranges of 139 k blocks
    (2, "mlp", 512, 16384, 2560),      # both products: 40 tiles of 256 rows, 20 column blocks
])
def test_tail_split_of_a_large_last_wave(pairs, kind, M, K, N):
    """A last wave above half of the units is cut into equal ranges of its k blocks: a unit ends one tile and starts
    the next."""
    prog, ins = _tail_case(kind, M, K, N, seed=M + N + pairs)
    try:
        dvm.set_matmul_cta_pairs(pairs)
        outs, _ = gpu_run(prog, ins)
        again, _ = gpu_run(prog, ins)
        dvm.set_matmul_tail_split(False)
        plain, _ = gpu_run(prog, ins)
    finally:
        dvm.set_matmul_tail_split(True)
        dvm.set_matmul_cta_pairs(1)
    want = oracle_run(prog, ins)
    check(prog, outs, want)
    check(prog, plain, want)
    assert not torch.isnan(outs[0].float()).any()
    assert torch.equal(outs[0], again[0])
    a, b = outs[0].float(), plain[0].float()
    assert (a - b).abs().max().item() <= 2.0 ** -7 * b.abs().max().item()
    assert (a != b).any().item()   # (the launch did split: some sums rounded differently)
