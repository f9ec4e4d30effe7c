"""GPU parity of the per-token dynamic activation path (Table 1, O1) against the CPU oracle, through
the C ABI: online per-token steps, rotate + quantize with one step per row, and the GEMM whose
epilogue applies the token's step."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import assert_bf16_close, assert_codes_tie_tolerant, rand_codes, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2410_05265_b200 import binding

    c = binding.Context()
    yield c
    c.check()
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("M,K,B,row_begin,clip", [(37, 4096, 4096, 4, 1.0), (19, 14336, 2048, 0, 0.9), (70, 256, 128, 1, 1.0),
                                                 (64, 128, 0, 0, 1.0), (3, 8192, 8192, 0, 0.75), (130, 1024, 512, 4, 1.0)])
def test_dynamic_scale_and_codes_match_oracle(ctx, M, K, B, row_begin, clip):
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin)
    x[M - 1] = 0  # an all-zero token
    s_ref = orc.dyn_act_scale(inputs.bits(x), B, clip, row_begin)
    s_gpu = torch.full((M,), -5.0, device="cuda")
    ctx.dyn_act_scale(x.cuda(), B, clip, row_begin, out=s_gpu)
    ctx.check()
    s = to_np(s_gpu)
    assert np.all(s[:row_begin] == -5.0), "prefix rows must not be written"
    live = np.arange(M) >= row_begin
    live[M - 1] = False
    assert np.all(np.abs(s[live] - s_ref[live]) <= 2e-6 * s_ref[live])
    assert s[M - 1] == 0.0 and s_ref[M - 1] == 1.0  # no step for an all-zero row: codes are zero under any
    # second pass with the GPU's own steps on both sides
    s_use = np.where(np.arange(M) < row_begin, 1.0, np.where(s == 0, 1.0, s)).astype(np.float32)
    ref, tie = orc.quant_act_rows(inputs.bits(x), B, s_use, row_begin, want_tie_dist=True)
    out = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act_rows(x.cuda(), B, s_gpu, row_begin, out=out)
    ctx.check()
    got = to_np(out)
    assert np.all(got[:row_begin] == 0x5A)
    n = assert_codes_tie_tolerant(got[row_begin:], ref[row_begin:], tie[row_begin:], "dynamic codes")
    # with the step tied to the row's own bf16 maximum, exact ties x / (max / 7) = k + 1/2 are common without a rotation
    assert n <= max(2, int((2e-4 if B else 2e-3) * x.numel()))
    assert np.all(got[M - 1] == 0)
    if clip == 1.0:  # every live token reaches the end of its range
        assert np.all(np.abs(orc.unpack_int4(got[live])).max(axis=1) == 7)


@pytest.mark.parametrize("M,K,B,row_begin,clip", [(37, 4096, 4096, 4, 1.0), (70, 2048, 2048, 0, 0.9), (5, 8192, 8192, 1, 0.75),
                                                 (19, 14336, 2048, 0, 0.9), (70, 256, 128, 1, 1.0), (300, 4096, 4096, 4, 1.0)])
def test_one_call_dynamic_quantizer_gives_the_bits_of_the_two_calls(ctx, M, K, B, row_begin, clip):
    """pq_dyn_hadamard_quant_act: one pass over the activations when a row is one wide transform block, the two
    passes otherwise; steps and codes equal those of pq_dyn_act_scale + pq_hadamard_quant_act_rows bit for bit
    (which the test above compares with the oracle), prefix rows untouched, an all-zero token included."""
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin)
    x[M - 1] = 0
    xd = x.cuda()
    s_two = torch.full((M,), -5.0, device="cuda")
    ctx.dyn_act_scale(xd, B, clip, row_begin, out=s_two)
    q_two = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act_rows(xd, B, s_two, row_begin, out=q_two)
    s_one = torch.full((M,), -5.0, device="cuda")
    q_one = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.dyn_hadamard_quant_act(xd, B, clip, row_begin, s_tok=s_one, out=q_one)
    ctx.check()
    assert torch.equal(s_one, s_two) and torch.equal(q_one, q_two)
    assert float(s_one[M - 1]) == 0.0 and int(q_one[M - 1].max()) == 0
    # and against the oracle's steps directly
    s_ref = orc.dyn_act_scale(inputs.bits(x), B, clip, row_begin)
    live = np.arange(M) >= row_begin
    live[M - 1] = False
    s = to_np(s_one)
    assert np.all(np.abs(s[live] - s_ref[live]) <= 2e-6 * s_ref[live])


def test_dynamic_path_is_scale_free_per_token(ctx):
    M, K = 24, 4096
    x = inputs.activations(M, K, seed=2)
    x2 = x.clone()
    x2[5] *= 16
    x2[9] *= 0.25
    xs = [t.cuda() for t in (x, x2)]
    s = [ctx.dyn_act_scale(t, K) for t in xs]
    q = [ctx.hadamard_quant_act_rows(t, K, si) for t, si in zip(xs, s)]
    ctx.check()
    assert torch.equal(q[0], q[1])
    assert float(s[1][5]) == 16 * float(s[0][5]) and float(s[1][9]) == 0.25 * float(s[0][9])


def _gemm_rows_case(ctx, M, N, K, seed, row_begin=0):
    rng = np.random.default_rng(seed)
    xq, wq = rand_codes(rng, M, K), rand_codes(rng, N, K)
    s_tok = (rng.random(M) * 0.05 + 0.002).astype(np.float32)
    s_w = (rng.random(N) * 0.004 + 0.001).astype(np.float32)
    acc_ref = orc.gemm_i4(xq, wq)
    out_ref = orc.dequant_bf16_rows(acc_ref, s_tok, s_w)
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a4_gemm_rows(dev(xq), dev(wq), dev(s_tok), dev(s_w), row_begin, out=out, acc_dbg=acc)
    ctx.check()
    acc = to_np(acc)
    assert np.all(acc[:row_begin] == -77) and np.all(to_np(out[:row_begin].float()) == 3.0)
    assert np.array_equal(acc[row_begin:], acc_ref[row_begin:])
    assert_bf16_close(inputs.bits(out)[row_begin:], out_ref[row_begin:], f"dynamic gemm {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [(1, 256, 128), (9, 96, 160), (16, 1024, 4096), (17, 96, 160), (257, 300, 1184), (300, 520, 4096),
                                   (130, 264, 14336), (600, 520, 8192)])
def test_gemm_rows_bit_exact_accumulators_and_per_token_epilogue(ctx, M, N, K):
    _gemm_rows_case(ctx, M, N, K, seed=M + N + K)


def test_gemm_rows_row_begin(ctx):
    _gemm_rows_case(ctx, 260, 256, 256, seed=11, row_begin=4)
    _gemm_rows_case(ctx, 12, 64, 256, seed=12, row_begin=4)


def test_dynamic_linear_end_to_end(ctx):
    M, K, N, P = 200, 4096, 1024, 4
    x = inputs.activations(M, K, seed=0, n_prefix=P)
    W = inputs.weights(N, K, seed=2)
    wq_ref, sw_ref = orc.quant_weights(inputs.bits(W))
    wq, s_w = ctx.quant_weights(W.cuda())
    s_tok = ctx.dyn_act_scale(x.cuda(), K, 1.0, P)
    xq = ctx.hadamard_quant_act_rows(x.cuda(), K, s_tok, P)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out = ctx.w4a4_gemm_rows(xq, wq, s_tok, s_w, P, acc_dbg=acc)
    ctx.check()
    s_np = to_np(s_tok)
    s_ref = orc.dyn_act_scale(inputs.bits(x), K, 1.0, P)
    assert np.all(np.abs(s_np[P:] - s_ref[P:]) <= 2e-6 * s_ref[P:])
    s_use = np.where(np.arange(M) < P, 1.0, s_np).astype(np.float32)
    xq_ref, tie = orc.quant_act_rows(inputs.bits(x), K, s_use, P, want_tie_dist=True)
    assert_codes_tie_tolerant(to_np(xq)[P:], xq_ref[P:], tie[P:], "dynamic chain codes")
    # the GPU's own codes and steps through the oracle GEMM and epilogue reproduce every row
    acc_ref = orc.gemm_i4(to_np(xq)[P:], wq_ref)
    assert np.array_equal(to_np(acc)[P:], acc_ref)
    assert_bf16_close(inputs.bits(out)[P:], orc.dequant_bf16_rows(acc_ref, s_np[P:], sw_ref), "dynamic chain output")
    # and the result approximates the unquantized product at least as well as one coarse static step does
    s_static = ctx.calib_act_scale(x.cuda(), K, P)
    out_static = ctx.w4a4_gemm(ctx.hadamard_quant_act(x.cuda(), K, s_static, P), wq, s_static, s_w, P)
    ref = (x.double() @ W.double().T)[P:]
    err_dyn = float((out[P:].double().cpu() - ref).pow(2).mean())
    err_sta = float((out_static[P:].double().cpu() - ref).pow(2).mean())
    assert err_dyn <= err_sta * 1.05


@pytest.mark.parametrize("M,K,B,row_begin,n_grid,lo,heavy", [(40, 1024, 1024, 4, 9, 0.2, True), (33, 6144, 2048, 0, 5, 0.5, False),
                                                            (64, 256, 0, 2, 16, 0.1, True), (5, 4096, 4096, 0, 1, 1.0, False),
                                                            (300, 512, 128, 0, 33, 0.25, True)])
def test_grid_search_for_the_shared_clipping_factor_matches_oracle(ctx, M, K, B, row_begin, n_grid, lo, heavy):
    """Sec. 3: the clipping factor shared by the tokens of per-token dynamic quantization, by squared error. Candidates,
    unclipped steps and every candidate's error against the oracle (whose step is gamma * max / 7 rounded once; the
    kernel's gamma * (max / 7) differs in the last bit at most, far inside the tolerance of the error sums), and the
    chosen factor: a candidate whose oracle error is the minimum up to that tolerance."""
    x = inputs.activations(M, K, seed=2, n_prefix=row_begin)
    if heavy:
        x[row_begin:, 5] *= 25.0                  # a far value in every row: clipping pays
    xb = inputs.bits(x)
    gamma, s_tok, cand, sse = ctx.grid_search_clip_dyn(x.cuda(), B, n_grid, lo, row_begin)
    ctx.check()
    g_ref, cand_ref, sse_ref = orc.grid_search_clip_dyn(xb, B, n_grid, lo, row_begin)
    assert np.array_equal(to_np(cand), cand_ref)
    assert np.allclose(to_np(s_tok)[row_begin:], orc.dyn_act_scale(xb, B, 1.0, row_begin)[row_begin:], rtol=2e-6)
    got = to_np(sse)
    assert np.allclose(got, sse_ref, rtol=2e-4, atol=1e-9), f"worst {np.max(np.abs(got - sse_ref) / np.maximum(sse_ref, 1e-30))}"
    pick = int(np.flatnonzero(cand_ref == float(gamma))[0])
    assert sse_ref[pick] <= sse_ref.min() * (1 + 4e-4) and got[pick] == got.min()
    assert sse_ref[pick] <= sse_ref[0], "never worse than no clipping"
    if heavy:
        assert pick != 0 and float(gamma) == float(g_ref)
    # the factor is what pq_dyn_act_scale takes: the quantizer run with it reproduces the searched error
    s_g = ctx.dyn_act_scale(x.cuda(), B, float(gamma), row_begin)
    codes = orc.unpack_int4(to_np(ctx.hadamard_quant_act_rows(x.cuda(), B, s_g, row_begin))).astype(np.float64)[row_begin:]
    y = orc.rotate_bf16(xb, B)[row_begin:]
    err = ((y - to_np(s_g).astype(np.float64)[row_begin:, None] * codes) ** 2).sum()
    assert err == pytest.approx(sse_ref[pick], rel=1e-3)
