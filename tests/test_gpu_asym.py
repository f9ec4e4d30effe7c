"""GPU parity of the activation quantizer of Eq. 1 as printed (asymmetric, zero point) against the CPU
oracle, through the C ABI: range calibration and max-min parameters, rotate + quantize with a zero point,
weight code sums, and the GEMM whose epilogue applies the zero-point correction."""
import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import TIE_WINDOW, assert_bf16_close, rand_codes, to_np

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


def gpu_codes(xq: torch.Tensor) -> np.ndarray:
    """Unsigned codes u from the packed signed nibbles the GPU stores (u - 8)."""
    return (orc.unpack_int4(to_np(xq)).astype(np.int32) + 8).astype(np.uint8)


def assert_u_tie_tolerant(got, ref, tie, what):
    g, r = got.astype(np.int32), ref.astype(np.int32)
    mism = g != r
    n = int(mism.sum())
    if n:
        assert np.all(np.abs(g[mism] - r[mism]) == 1), f"{what}: a code differs by more than one"
        assert np.all(tie[mism] < TIE_WINDOW), f"{what}: mismatch away from a tie"
    return n


@pytest.mark.parametrize("M,K,B,row_begin,shift", [(37, 4096, 4096, 4, 0.0), (19, 14336, 2048, 0, 0.0), (70, 256, 128, 1, 0.0),
                                                  (64, 128, 0, 0, 3.0), (64, 256, 0, 2, -2.5), (3, 8192, 8192, 0, 0.0)])
def test_asym_calibration_and_codes_match_oracle(ctx, M, K, B, row_begin, shift):
    x = (inputs.activations(M, K, seed=0, n_prefix=row_begin).float() + shift).to(torch.bfloat16)
    cal = (inputs.activations(max(M, 16), K, seed=1, n_prefix=row_begin).float() + shift).to(torch.bfloat16)
    mn, mx = orc.calib_act_minmax(inputs.bits(cal), B, row_begin)
    s_ref, z_ref = orc.asym_params(mn, mx)
    s_gpu, z_gpu = ctx.calib_act_asym(cal.cuda(), B, row_begin)
    ctx.check()
    s, z = float(s_gpu), int(z_gpu)
    assert abs(s - float(s_ref)) <= 4e-6 * float(s_ref) and abs(z - z_ref) <= 1
    if shift > 0 and B == 0:
        assert z < 8, "a positive offset moves the zero point down"
    if shift < 0 and B == 0:
        assert z > 8
    # quantize with the GPU's own parameters on both sides
    ref, tie = orc.quant_act_asym(inputs.bits(x), B, np.float32(s), z, row_begin, want_tie_dist=True)
    out = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act_asym(x.cuda(), B, s_gpu, z_gpu, row_begin, out=out)
    ctx.check()
    assert np.all(to_np(out)[:row_begin] == 0x5A), "prefix rows must not be written"
    n = assert_u_tie_tolerant(gpu_codes(out)[row_begin:], ref[row_begin:], tie[row_begin:], "asymmetric codes")
    # without a rotation the bf16 inputs sit on a coarse grid and the step comes from two of them: exact ties are common
    assert n <= max(2, int((2e-4 if B else 1e-2) * x.numel()))
    # the calibration batch itself fills the whole code range
    cq = gpu_codes(ctx.hadamard_quant_act_asym(cal.cuda(), B, s_gpu, z_gpu, row_begin))[row_begin:]
    assert cq.min() == 0 and cq.max() >= 14


def test_asym_params_match_oracle_bit_for_bit_on_exact_ranges(ctx):
    """No rotation and exactly representable data: the GPU sees the same minimum and maximum as the oracle, so the
    step and the zero point must agree bit for bit."""
    for lo, hi in [(-1.0, 2.75), (0.0, 15.0), (-15.0, 0.0), (-3.5, 0.25), (2.0, 2.0), (0.125, 7.0)]:
        x = torch.full((4, 128), lo, dtype=torch.bfloat16)
        x[1, 5] = hi
        s_ref, z_ref = orc.asym_params(lo, hi)
        s_gpu, z_gpu = ctx.calib_act_asym(x.cuda(), 0)
        assert float(s_gpu) == float(s_ref) and int(z_gpu) == z_ref, (lo, hi)
    ctx.check()


def test_weight_code_sums_match_numpy(ctx):
    rng = np.random.default_rng(3)
    for N, K in [(5, 8), (300, 4096), (17, 14336), (64, 160)]:
        wq = rand_codes(rng, N, K)
        got = to_np(ctx.weight_code_sums(dev(wq)))
        assert np.array_equal(got, orc.unpack_int4(wq).astype(np.int64).sum(1))
    lo = np.full((3, 65536 // 2), 0x88, np.uint8)
    assert np.all(to_np(ctx.weight_code_sums(dev(lo))) == -8 * 65536)
    ctx.check()


def _gemm_asym_case(ctx, M, N, K, z, seed, row_begin=0):
    rng = np.random.default_rng(seed)
    u = rng.integers(0, 16, (M, K)).astype(np.uint8)
    xq = orc.pack_int4((u.astype(np.int32) - 8).astype(np.int8))
    wq = rand_codes(rng, N, K)
    s_a = np.float32(0.0173)
    s_w = (rng.random(N) * 0.004 + 0.001).astype(np.float32)
    acc_ref = orc.gemm_asym(u, z, wq)
    out_ref = orc.dequant_bf16(acc_ref, s_a, s_w)
    wsum = ctx.weight_code_sums(dev(wq))
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a4_gemm_asym(dev(xq), dev(wq), torch.tensor([s_a], device="cuda"), torch.tensor([z], dtype=torch.int32, device="cuda"),
                       dev(s_w), wsum, row_begin, out=out, acc_dbg=acc)
    ctx.check()
    acc = to_np(acc)
    assert np.all(acc[:row_begin] == -77) and np.all(to_np(out[:row_begin].float()) == 3.0)
    assert np.array_equal(acc[row_begin:], acc_ref[row_begin:]), "sum (u - z) w must be bit-exact"
    assert_bf16_close(inputs.bits(out)[row_begin:], out_ref[row_begin:], f"asym gemm {M}x{N}x{K} z={z}")


@pytest.mark.parametrize("M,N,K,z", [(1, 256, 128, 3), (9, 96, 160, 15), (16, 1024, 4096, 0), (17, 96, 160, 8), (257, 300, 1184, 5),
                                     (300, 520, 4096, 11), (130, 264, 14336, 2), (600, 520, 8192, 13)])
def test_gemm_asym_bit_exact(ctx, M, N, K, z):
    _gemm_asym_case(ctx, M, N, K, z, seed=M + N + K)


def test_gemm_asym_row_begin_and_many_tiles(ctx):
    _gemm_asym_case(ctx, 260, 256, 256, 6, seed=11, row_begin=4)
    _gemm_asym_case(ctx, 12, 64, 256, 9, seed=12, row_begin=4)
    _gemm_asym_case(ctx, 1024, 5120, 256, 4, seed=5)


def test_gemm_asym_zero_point_8_is_the_symmetric_gemm(ctx):
    rng = np.random.default_rng(1)
    M, N, K = 40, 512, 1024
    xq, wq = rand_codes(rng, M, K), rand_codes(rng, N, K)
    s_a, s_w = torch.tensor([0.01], device="cuda"), torch.full((N,), 0.002, device="cuda")
    z8 = torch.tensor([8], dtype=torch.int32, device="cuda")
    a = ctx.w4a4_gemm_asym(dev(xq), dev(wq), s_a, z8, s_w, ctx.weight_code_sums(dev(wq)))
    b = ctx.w4a4_gemm(dev(xq), dev(wq), s_a, s_w)
    ctx.check()
    assert torch.equal(a, b)


def test_asym_linear_end_to_end_beats_symmetric_on_offset_activations(ctx):
    """calibrate -> quantize -> GEMM on activations with a large positive offset (what a zero point is for): the GPU's
    own codes through the oracle reproduce it exactly, and the error against the unquantized product is smaller than
    with the symmetric quantizer."""
    M, K, N = 160, 1024, 512
    x = (inputs.activations(M, K, seed=0).float().abs() * 0.5 + 1.0).to(torch.bfloat16)   # strictly positive rows
    W = inputs.weights(N, K, seed=2)
    wq_ref, sw_ref = orc.quant_weights(inputs.bits(W))
    wq, s_w = ctx.quant_weights(W.cuda())
    wsum = ctx.weight_code_sums(wq)
    s_a, z_a = ctx.calib_act_asym(x.cuda(), 0)
    xq = ctx.hadamard_quant_act_asym(x.cuda(), 0, s_a, z_a)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out = ctx.w4a4_gemm_asym(xq, wq, s_a, z_a, s_w, wsum, acc_dbg=acc)
    ctx.check()
    z = int(z_a)
    assert z == 0 or z < 8
    acc_ref = orc.gemm_asym(gpu_codes(xq), z, wq_ref)
    assert np.array_equal(to_np(acc), acc_ref)
    assert_bf16_close(inputs.bits(out), orc.dequant_bf16(acc_ref, np.float32(float(s_a)), sw_ref), "asym chain output")
    ref = x.double() @ W.double().T
    s_sym = ctx.calib_act_scale(x.cuda(), 0)
    out_sym = ctx.w4a4_gemm(ctx.hadamard_quant_act(x.cuda(), 0, s_sym), wq, s_sym, s_w)
    err_asym = float((out.double().cpu() - ref).pow(2).mean())
    err_sym = float((out_sym.double().cpu() - ref).pow(2).mean())
    assert err_asym < 0.6 * err_sym


@pytest.mark.parametrize("M,K,B,row_begin,n_grid,lo,outlier", [(40, 1024, 1024, 4, 6, 0.3, 0.0), (33, 6144, 2048, 0, 4, 0.5, 0.0),
                                                              (64, 256, 0, 2, 8, 0.2, 60.0), (5, 4096, 4096, 0, 1, 1.0, 0.0),
                                                              (17, 128, 128, 0, 16, 0.1, 0.0)])
def test_grid_search_for_s_and_z_matches_oracle(ctx, M, K, B, row_begin, n_grid, lo, outlier):
    """The n x n candidates against the oracle's (from the oracle's own range), the squared error of every candidate
    against the oracle's error of the same (s, z), and the chosen pair: one whose oracle error is the minimum up to
    the tolerance of the comparison (near-equal candidates may swap places in fp32)."""
    x = inputs.activations(M, K, seed=1, n_prefix=row_begin)
    if outlier:
        x[row_begin + 1, 7] = outlier          # a far value in an ordinary row: clipping it pays
    xb = inputs.bits(x)
    s_a, z_a, cand_s, cand_z, sse = ctx.grid_search_act_asym(x.cuda(), B, n_grid, lo, row_begin)
    ctx.check()
    cs, cz, got = to_np(cand_s), to_np(cand_z), to_np(sse)
    mn, mx = orc.calib_act_minmax(xb, B, row_begin)
    cs_ref, cz_ref = orc.grid_candidates(mn, mx, n_grid, lo)
    assert np.allclose(cs, cs_ref, rtol=4e-6) and np.all(np.abs(cz - cz_ref) <= 1)
    assert (cs[0], cz[0]) == tuple(float(v) if i == 0 else int(v) for i, v in enumerate(ctx.calib_act_asym(x.cuda(), B, row_begin)))
    ref = np.array([orc.quant_sse_asym(xb, B, cs[c], int(cz[c]), row_begin) for c in range(n_grid * n_grid)])
    assert np.allclose(got, ref, rtol=2e-4, atol=1e-9), f"worst {np.max(np.abs(got - ref) / np.maximum(ref, 1e-30))}"
    pick = [c for c in range(len(cs)) if cs[c] == float(s_a) and cz[c] == int(z_a)]
    assert pick, "the result is one of the candidates"
    assert ref[pick[0]] <= ref.min() * (1 + 4e-4) and got[pick[0]] == got.min()
    assert ref[pick[0]] <= ref[0], "never worse than the max-min pair"
    if outlier:
        assert pick[0] != 0 and ref[pick[0]] < 0.7 * ref[0]
