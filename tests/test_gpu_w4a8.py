"""GPU parity of the W4A8 linear layer (8-bit static per-tensor activation codes, Sec. 5.1) against
the CPU oracle, through the C ABI: rotate + quantize to one signed byte per element, the int8 x int4
GEMM with exact int32 accumulators, and the chain of both."""
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


def assert_codes8_tie_tolerant(got: np.ndarray, ref: np.ndarray, tie: np.ndarray, what: str) -> int:
    """int8 codes equal the oracle's except within TIE_WINDOW of a rounding tie, where they may differ by one."""
    g, r = got.astype(np.int32), ref.astype(np.int32)
    mism = g != r
    n = int(mism.sum())
    if n:
        assert np.all(np.abs(g[mism] - r[mism]) == 1), f"{what}: a code differs by more than one"
        assert np.all(tie[mism] < TIE_WINDOW), f"{what}: mismatch away from a tie (max dist {tie[mism].max()})"
    return n


@pytest.mark.parametrize("M,K,B,row_begin", [(37, 4096, 4096, 4), (19, 14336, 2048, 0), (5, 256, 128, 1), (64, 128, 0, 0),
                                            (3, 8192, 8192, 0), (130, 1024, 512, 4)])
def test_hadamard_quant_act8_matches_oracle(ctx, M, K, B, row_begin):
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin)
    cal = inputs.activations(max(M, 16), K, seed=1, n_prefix=row_begin)
    s_ref = orc.calib_act_scale8(inputs.bits(cal), B, row_begin)
    s_gpu = ctx.calib_act_scale8(cal.cuda(), B, row_begin)
    ctx.check()
    assert abs(float(s_gpu[0]) - float(s_ref)) <= 2e-6 * float(s_ref)
    s_a = torch.tensor([s_ref], dtype=torch.float32, device="cuda")
    ref, tie = orc.quant_act8(inputs.bits(x), B, s_ref, row_begin, want_tie_dist=True)
    out = torch.full((M, K), 0x5A, dtype=torch.int8, device="cuda")
    ctx.hadamard_quant_act8(x.cuda(), B, s_a, row_begin, out=out)
    ctx.check()
    got = to_np(out)
    assert np.all(got[:row_begin] == 0x5A), "prefix rows must not be written"
    n = assert_codes8_tie_tolerant(got[row_begin:], ref[row_begin:], tie[row_begin:], "hadamard_quant_act8")
    assert n <= max(2, int(2e-3 * x.numel()))  # 18 times finer steps than 4-bit: ties are that much more frequent
    assert np.abs(got[row_begin:].astype(int)).max() >= 100, "the calibrated step must use the 8-bit range"


def test_quant_act8_clamps_at_both_ends(ctx):
    K = 128
    x = torch.zeros((2, K), dtype=torch.bfloat16)
    x[0, :] = torch.linspace(-80, 80, K)
    x[1, ::2] = 1e4
    x[1, 1::2] = -1e4
    s_a = torch.tensor([0.25], device="cuda")
    got = to_np(ctx.hadamard_quant_act8(x.cuda(), 0, s_a))
    ctx.check()
    ref = orc.quant_act8(inputs.bits(x), 0, 0.25)
    assert np.array_equal(got, ref) and got.min() == -128 and got.max() == 127


def _gemm8_case(ctx, M, N, K, seed, row_begin=0):
    rng = np.random.default_rng(seed)
    xq8 = rng.integers(-128, 128, (M, K)).astype(np.int8)
    wq = rand_codes(rng, N, K)
    s_a = np.float32(0.00137)
    s_w = (rng.random(N) * 0.004 + 0.001).astype(np.float32)
    acc_ref = orc.gemm_i8i4(xq8, wq)
    out_ref = orc.dequant_bf16(acc_ref, s_a, s_w)
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a8_gemm(dev(xq8), dev(wq), torch.tensor([s_a], device="cuda"), dev(s_w), row_begin, out=out, acc_dbg=acc)
    ctx.check()
    acc = to_np(acc)
    assert np.all(acc[:row_begin] == -77) and np.all(to_np(out[:row_begin].float()) == 3.0)
    assert np.array_equal(acc[row_begin:], acc_ref[row_begin:]), "int32 accumulators must be bit-exact"
    assert_bf16_close(inputs.bits(out)[row_begin:], out_ref[row_begin:], f"w4a8 gemm {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [(1, 256, 128), (17, 96, 160), (256, 256, 128), (257, 300, 1184), (300, 520, 4096),
                                   (512, 264, 2048), (40, 4096, 512)])
def test_w4a8_gemm_bit_exact(ctx, M, N, K):
    _gemm8_case(ctx, M, N, K, seed=M + N + K)


@pytest.mark.parametrize("M", [1, 4, 8, 9, 16])
@pytest.mark.parametrize("N,K", [(48, 4096), (1024, 4096), (40, 160), (4096, 14336)])
def test_w4a8_gemm_decode_shapes_bit_exact(ctx, M, N, K):
    """Up to 16 tokens: the weight-streaming kernel with s8 activation codes."""
    if N * K > 1 << 24 and M not in (1, 16):
        pytest.skip("large shape covered at M=1 and M=16")
    _gemm8_case(ctx, M, N, K, seed=M * 7 + N)
    if M == 9:
        _gemm8_case(ctx, M + 4, N, K, seed=N, row_begin=4)


@pytest.mark.parametrize("M,K,B,row_begin,N", [(70, 6144, 2048, 4, 264), (33, 4096, 4096, 0, 96), (9, 8192, 8192, 1, 40),
                                               (37, 768, 256, 0, 64), (21, 384, 0, 2, 48), (300, 4096, 4096, 4, 520)])
def test_four_bit_codes_one_per_byte_give_the_packed_path_bit_for_bit(ctx, M, K, B, row_begin, N):
    """pq_hadamard_quant_act_c8: the codes of pq_hadamard_quant_act (which the parity tests compare with the oracle),
    unpacked; pq_w4a8_gemm on them returns the sums and outputs of pq_w4a4_gemm on the packed codes."""
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin).cuda()
    s_a = ctx.calib_act_scale(x, B, row_begin)
    packed = ctx.hadamard_quant_act(x, B, s_a, row_begin)
    bytes8 = torch.full((M, K), 0x5A, dtype=torch.int8, device="cuda")
    ctx.hadamard_quant_act_c8(x, B, s_a, row_begin, out=bytes8)
    ctx.check()
    assert np.all(to_np(bytes8)[:row_begin] == 0x5A), "prefix rows must not be written"
    assert np.array_equal(to_np(bytes8)[row_begin:], orc.unpack_int4(to_np(packed))[row_begin:])
    wq = dev(rand_codes(np.random.default_rng(M + N), N, K))
    s_w = torch.full((N,), 0.003, device="cuda")
    acc4 = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    acc8 = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out4 = ctx.w4a4_gemm(packed, wq, s_a, s_w, row_begin, acc_dbg=acc4)
    out8 = ctx.w4a8_gemm(bytes8, wq, s_a, s_w, row_begin, acc_dbg=acc8)
    ctx.check()
    assert torch.equal(acc4[row_begin:], acc8[row_begin:]) and torch.equal(out4[row_begin:], out8[row_begin:])


def test_w4a8_gemm_many_tiles_and_row_begin(ctx):
    _gemm8_case(ctx, 1024, 5120, 256, seed=5)       # 80 tiles on 74 CTA pairs: some pairs take a second tile
    _gemm8_case(ctx, 260, 256, 256, seed=11, row_begin=4)


def test_w4a8_gemm_extreme_codes_fit_int32(ctx):
    M, N, K = 128, 256, 28672
    xq8 = np.full((M, K), -128, np.int8)
    wq = np.full((N, K // 2), 0x88, np.uint8)  # every weight code -8
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    ctx.w4a8_gemm(dev(xq8), dev(wq), torch.ones(1, device="cuda"), torch.ones(N, device="cuda"), acc_dbg=acc)
    ctx.check()
    assert int(acc.min()) == int(acc.max()) == 1024 * K


def test_w4a8_linear_end_to_end(ctx):
    """calibrate -> rotate + quantize -> GEMM against the oracle chain; rows whose codes all match the
    oracle's must give bit-exact accumulators."""
    M, K, N = 192, 4096, 1024
    x = inputs.activations(M, K, seed=0)
    cal = inputs.activations(M, K, seed=1)
    W = inputs.weights(N, K, seed=2)
    s_ref = orc.calib_act_scale8(inputs.bits(cal), K)
    xq_ref, tie = orc.quant_act8(inputs.bits(x), K, s_ref, want_tie_dist=True)
    wq_ref, sw_ref = orc.quant_weights(inputs.bits(W))
    acc_ref = orc.gemm_i8i4(xq_ref, wq_ref)
    s_a = torch.tensor([s_ref], device="cuda")
    wq, s_w = ctx.quant_weights(W.cuda())
    xq8 = ctx.hadamard_quant_act8(x.cuda(), K, s_a)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out = ctx.w4a8_gemm(xq8, wq, s_a, s_w, acc_dbg=acc)
    ctx.check()
    assert np.array_equal(to_np(wq), wq_ref)
    assert_codes8_tie_tolerant(to_np(xq8), xq_ref, tie, "w4a8 chain codes")
    clean = ~(to_np(xq8) != xq_ref).any(axis=1)
    assert clean.sum() >= M // 2
    assert np.array_equal(to_np(acc)[clean], acc_ref[clean])
    out_ref = orc.dequant_bf16(acc_ref, s_ref, sw_ref)
    assert_bf16_close(inputs.bits(out)[clean], out_ref[clean], "w4a8 chain output")
    # the GPU's own codes through the oracle GEMM reproduce every row
    assert np.array_equal(to_np(acc), orc.gemm_i8i4(to_np(xq8), wq_ref))


@pytest.mark.parametrize("name,N,K", [("gate|up", 28672, 4096), ("down", 4096, 14336)])
def test_w4a8_gemm_llama8b_prefill_2048_sampled_rows(ctx, name, N, K):
    M, P = 2048, 4
    g = torch.Generator(device="cuda").manual_seed(N + K)
    xq8 = torch.randint(-128, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
    wq = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    s_a = torch.tensor([0.00137], device="cuda")
    s_w = torch.rand(N, device="cuda", generator=g) * 0.004 + 0.001
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a8_gemm(xq8, wq, s_a, s_w, P, out=out, acc_dbg=acc)
    ctx.check()
    assert int(acc[:P].min()) == int(acc[:P].max()) == -77
    rng = np.random.default_rng(N)
    rows = np.unique(np.concatenate([[P, M - 1, 127 + P, 128 + P, 255, 256], rng.integers(P, M, 8)]))
    acc_ref = orc.gemm_i8i4(to_np(xq8[rows]), to_np(wq))
    assert np.array_equal(to_np(acc[rows]), acc_ref), "sampled accumulator rows must be bit-exact"
    assert_bf16_close(inputs.bits(out[rows]), orc.dequant_bf16(acc_ref, np.float32(0.00137), to_np(s_w)), f"w4a8 gemm {name}")
    out2 = torch.full_like(out, 3.0)
    ctx.w4a8_gemm(xq8, wq, s_a, s_w, P, out=out2)
    ctx.check()
    assert torch.equal(out2, out)
