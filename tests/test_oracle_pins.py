"""Pins for the CPU oracle: it is checked against closed forms, invariants, brute force and
independent library routines before anything is compared with it. No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from scipy.linalg import hadamard

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    return np.loadtxt(os.path.join(GOLDEN, name), comments="#")


def bf16_bits(x):
    return inputs.bits(torch.as_tensor(np.asarray(x, np.float64)).to(torch.bfloat16))


def fp16_bits(x):
    return inputs.bits(torch.as_tensor(np.asarray(x, np.float64)).to(torch.float16))


rng = np.random.default_rng(1234)


# ---------------------------------------------------------------- formats
def test_bf16_roundtrip_matches_library_rounding():
    x = np.concatenate([rng.standard_normal(4000) * np.exp(rng.standard_normal(4000) * 8), [0.0, -0.0, 1e-40, 3e38]])
    # exact ties between two bf16 neighbours must go to even
    ties = np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, -(2.0 + 2.0**-7), 2.0**-130 + 2.0**-134])
    x = np.concatenate([x, ties])
    got = orc.f64_to_bf16(x)
    # torch rounds float64 -> bf16 through float32; avoid that double rounding in the reference by
    # using values whose float32 image is exact or far from a bf16 tie
    ref = inputs.bits(torch.from_numpy(x).to(torch.float32).to(torch.bfloat16))
    f32_exact = x.astype(np.float32).astype(np.float64) == x
    assert np.array_equal(got[f32_exact], ref[f32_exact])
    assert np.mean(got == ref) > 0.999
    assert got[-4] == 0x3F80 and got[-3] == 0x3F82  # 1+2^-8 -> 1.0 (even), 1+3*2^-8 -> 1+2^-6
    back = orc.bf16_to_f64(got)
    assert np.array_equal(orc.f64_to_bf16(back), got)


def test_fp16_decode_matches_numpy_for_every_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    ref = allbits.view(np.float16).astype(np.float64)
    got = orc.fp16_to_f64(allbits)
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok], ref[ok]) and np.all(np.isnan(got[~ok]))


def test_pack_layout_low_nibble_first_twos_complement():
    assert orc.unpack_int4(np.array([[0x21]], np.uint8)).tolist() == [[1, 2]]
    assert orc.unpack_int4(np.array([[0xF8]], np.uint8)).tolist() == [[-8, -1]]
    every = np.arange(256, dtype=np.uint8).reshape(16, 16)
    codes = orc.unpack_int4(every)
    assert codes.min() == -8 and codes.max() == 7
    assert np.array_equal(orc.pack_int4(codes), every)
    lo = (every & 0xF).astype(np.int16)
    hi = (every >> 4).astype(np.int16)
    assert np.array_equal(codes[:, 0::2], np.where(lo >= 8, lo - 16, lo))
    assert np.array_equal(codes[:, 1::2], np.where(hi >= 8, hi - 16, hi))


# ---------------------------------------------------------------- rotation (App. B)
def test_hadamard_golden_h4():
    H4 = _load("hadamard_h4_sylvester.txt")
    got = orc.rotate_f64(np.eye(4), 4) * 2.0
    assert np.array_equal(got, H4)


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_hadamard_orthogonality(n):
    H = orc.rotate_f64(np.eye(n), n) * math.sqrt(n)
    H = np.rint(H)
    assert set(np.unique(H).tolist()) <= {-1.0, 1.0}
    assert np.array_equal(H @ H.T, n * np.eye(n))
    assert np.array_equal(H, H.T)


@pytest.mark.parametrize("n", [2, 8, 64, 256])
def test_rotation_equals_library_sylvester_product(n):
    x = rng.standard_normal((5, n))
    ref = x @ hadamard(n).astype(np.float64) / math.sqrt(n)
    assert np.allclose(orc.rotate_f64(x, n), ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("n", [2048, 4096])
def test_rotation_large_blocks(n):
    x = rng.standard_normal((3, n))
    y = orc.rotate_f64(x, n)
    ref = x @ hadamard(n).astype(np.float64) / math.sqrt(n)
    assert np.allclose(y, ref, rtol=0, atol=1e-10)
    # unit vector -> one matrix row; all-ones -> sqrt(n) * e_0
    e = np.zeros((1, n))
    e[0, 37] = 1.0
    col = orc.rotate_f64(e, n)[0] * math.sqrt(n)
    i = np.arange(n)
    parity = np.array([bin(v & 37).count("1") & 1 for v in i])
    assert np.array_equal(np.rint(col), np.where(parity == 1, -1.0, 1.0))
    ones = orc.rotate_f64(np.ones((1, n)), n)[0]
    assert abs(ones[0] - math.sqrt(n)) < 1e-12 and np.all(ones[1:] == 0.0)


def test_rotation_involution_and_parseval():
    x = rng.standard_normal((4, 512))
    y = orc.rotate_f64(x, 512)
    assert np.allclose(orc.rotate_f64(y, 512), x, atol=1e-12)
    assert np.allclose((y**2).sum(1), (x**2).sum(1), rtol=1e-12)


def test_block_diagonal_rotation_is_independent_per_block():
    x = rng.standard_normal((3, 7 * 64))
    y = orc.rotate_f64(x, 64)
    for b in range(7):
        assert np.array_equal(y[:, b * 64:(b + 1) * 64], orc.rotate_f64(np.ascontiguousarray(x[:, b * 64:(b + 1) * 64]), 64))
    assert np.array_equal(orc.rotate_f64(x, 0), x)


def test_rotate_bf16_decodes_bits_exactly():
    xb = bf16_bits(rng.standard_normal((4, 128)))
    assert np.array_equal(orc.rotate_bf16(xb, 128), orc.rotate_f64(orc.bf16_to_f64(xb), 128))


def test_computational_invariance_of_rotation():
    # App. B: rotating activations and counter-rotating weights leaves x W^T unchanged
    n = 256
    x = rng.standard_normal((6, n))
    W = rng.standard_normal((10, n))
    lhs = orc.rotate_f64(x, n) @ orc.rotate_f64(W, n).T
    assert np.allclose(lhs, x @ W.T, rtol=0, atol=1e-11)


# ---------------------------------------------------------------- quantizer (Eq. 1)
def test_quantizer_golden_worked_example():
    g = _load("quantizer_eq1_worked.txt")
    codes = orc.quant_f64(g[:, 0], 0.25)
    assert codes.tolist() == g[:, 2].astype(int).tolist()
    assert (np.clip(codes.astype(int) + 8, 0, 15)).tolist() == g[:, 3].astype(int).tolist()


def test_quantizer_range_ties_clamp_monotone_idempotent():
    v = np.linspace(-3.0, 3.0, 4001)
    c = orc.quant_f64(v, 0.25)
    assert c.min() == -8 and c.max() == 7
    assert np.all(np.diff(c.astype(int)) >= 0)
    ties = (np.arange(-8, 7) + 0.5) * 0.25
    ct = orc.quant_f64(ties, 0.25).astype(int)
    assert np.all(ct % 2 == 0), "ties must go to the even code"
    assert np.all(np.abs(ct - (np.arange(-8, 7) + 0.5)) == 0.5)
    deq = c.astype(np.float64) * 0.25
    assert np.array_equal(orc.quant_f64(deq, 0.25), c)
    inside = np.abs(v) <= 1.75
    assert np.all(np.abs(deq[inside] - v[inside]) <= 0.125 + 1e-15)


def test_quant_act_codes_and_tie_distance():
    K = 64
    x = rng.standard_normal((5, K))
    xb = bf16_bits(x)
    y = orc.rotate_bf16(xb, K)
    s = np.float32(np.abs(y).max() / 7)
    xq, tie = orc.quant_act(xb, K, s, want_tie_dist=True)
    codes = orc.unpack_int4(xq)
    r = y / np.float64(s)
    assert np.all(np.abs(codes - r) <= 0.5 + 1e-12)
    assert np.abs(codes).max() == 7
    frac = r - np.floor(r)
    assert np.allclose(tie, np.abs(frac - 0.5), atol=1e-6)
    # rows below row_begin are left untouched
    xq2 = orc.quant_act(xb, K, s, row_begin=2)
    assert np.all(xq2[:2] == 0) and np.array_equal(xq2[2:], xq[2:])


def test_static_scale_ignores_prefixed_rows():
    M, K, P = 12, 128, 4
    x = inputs.activations(M, K, seed=1, n_prefix=P)
    xb = inputs.bits(x)
    y = orc.rotate_bf16(xb, K)
    s = orc.calib_act_scale(xb, K, row_begin=P)
    assert s == np.float32(np.abs(y[P:].astype(np.float32)).max() / 7.0)
    x2 = x.clone()
    x2[:P] *= 1000.0
    assert orc.calib_act_scale(inputs.bits(x2), K, row_begin=P) == s
    assert orc.calib_act_scale(xb, K, row_begin=0) > 10 * s  # with the outlier rows the scale explodes


# ---------------------------------------------------------------- weights (RTN per output channel)
def test_weight_quantization_rtn_per_channel():
    W = inputs.weights(24, 96, seed=2)
    W[5] = 0
    Wb = inputs.bits(W)
    wq, s_w = orc.quant_weights(Wb)
    Wf = W.to(torch.float32).numpy()
    mx = np.abs(Wf).max(1)
    expect = np.where(mx == 0, np.float32(1), mx / np.float32(7)).astype(np.float32)
    assert np.array_equal(s_w, expect)
    codes = orc.unpack_int4(wq).astype(np.int32)
    assert codes.min() >= -7 and codes.max() <= 7  # symmetric max/7 never needs -8
    assert np.all(codes[5] == 0) and s_w[5] == 1.0
    am = np.abs(Wf).argmax(1)
    rows = np.arange(24)
    assert np.all(np.abs(codes[rows, am])[mx > 0] == 7)
    assert np.all(np.abs(codes * s_w[:, None].astype(np.float64) - Wf) <= s_w[:, None] * 0.5 * (1 + 1e-6))
    # idempotent: quantizing the dequantized weights (exact in bf16 only approximately, so use codes*2^-k scale)
    W2 = (np.arange(-7, 8)[None, :].repeat(3, 0) * 0.25).astype(np.float64)
    wq2, s2 = orc.quant_weights(bf16_bits(np.concatenate([W2, W2[:, :1]], 1)))
    assert np.array_equal(orc.unpack_int4(wq2)[:, :15], np.arange(-7, 8)[None, :].repeat(3, 0)) and np.all(s2 == 0.25)


def _rne_codes_f64(x, s, lo=-8, hi=7):
    """clamp(round_half_even(x / s)) with the quotient in float64 (numpy's rint rounds half to even)."""
    return np.clip(np.rint(x.astype(np.float64) / s.astype(np.float64)), lo, hi).astype(np.int64)


def test_weight_quantizer_tie_direction_and_fp32_decision():
    # exact ties: a row whose maximum is 1.75 has step 1.75 / 7 = 0.25 exactly; the elements (k + 1/2) / 4 are
    # bf16 numbers whose quotient is exactly k + 1/2. Half-even sends them to the even neighbour, both signs.
    ks = np.arange(-7, 7)
    row = np.concatenate([(ks + 0.5) * 0.25, [1.75, -1.75]])
    wq, s_w, tie = orc.quant_weights(bf16_bits(row[None, :]), want_tie_dist=True)
    codes = orc.unpack_int4(wq)[0]
    assert s_w[0] == 0.25 and np.all(tie[0, :14] == 0.0) and np.all(tie[0, 14:] == 0.5)
    want = np.where(ks % 2 == 0, ks, ks + 1)  # k + 1/2 -> the even one of k, k + 1
    assert codes[:14].tolist() == want.tolist() and codes[14:].tolist() == [7, -7]
    assert codes[ks.tolist().index(0)] == 0 and codes[ks.tolist().index(-1)] == 0 and codes[ks.tolist().index(1)] == 2
    # the fp32 decision equals the double-precision one except next to a tie: on the synthetic weights every
    # differing code sits within 1e-4 of a tie and differs by exactly one, and such cases are rare
    W = inputs.weights(64, 4096, seed=2)
    wq, s_w, tie = orc.quant_weights(inputs.bits(W), want_tie_dist=True)
    got = orc.unpack_int4(wq).astype(np.int64)
    ref = _rne_codes_f64(W.to(torch.float64).numpy(), s_w[:, None])
    diff = got != ref
    assert np.all(tie[diff] < 1e-4) and np.all(np.abs(got - ref)[diff] == 1)
    assert diff.sum() <= 1e-3 * diff.size, diff.sum()  # bf16 inputs over a max/7 step land next to ties often
    # away from ties nothing is left to the precision: the code is the nearest integer of the exact quotient
    far = tie > 1e-4
    r = W.to(torch.float64).numpy() / s_w[:, None].astype(np.float64)
    assert np.all(np.abs(got - r)[far] < 0.5)


def test_kv_quantizer_tie_direction_and_fp32_decision():
    # exact ties with a power-of-two step, k even and odd, both signs; beyond +-7.5 steps the code clamps
    B, T, H, D, Tmax = 1, 1, 1, 16, 2
    ks = np.arange(-8, 8)
    kvals = (ks + 0.5) * 0.25          # k + 1/2 for k = -8 .. 7: -7.5 .. 7.5 steps
    vvals = (ks + 0.5) * 2.0
    kb, vb = bf16_bits(kvals.reshape(B, T, H, D)), bf16_bits(vvals.reshape(B, T, H, D))
    kq, vq = np.zeros((B, H, Tmax, D // 2), np.uint8), np.zeros((B, H, Tmax, D // 2), np.uint8)
    tie_k, tie_v = np.ones((B, T, H, D), np.float32), np.ones((B, T, H, D), np.float32)
    length = np.zeros(B, np.int32)
    assert orc.kv4_append(kb, vb, np.array([0.25], np.float32), np.array([2.0], np.float32), kq, vq, length, tie_k, tie_v) == 0
    want = np.clip(np.where(ks % 2 == 0, ks, ks + 1), -8, 7)
    assert orc.unpack_int4(kq)[0, 0, 0].tolist() == want.tolist() == [-8, -6, -6, -4, -4, -2, -2, 0, 0, 2, 2, 4, 4, 6, 6, 7]
    assert orc.unpack_int4(vq)[0, 0, 0].tolist() == want.tolist()
    assert np.all(tie_k == 0.0) and np.all(tie_v == 0.0)
    # fp32-decided codes against the double-precision decision on the synthetic K/V with max/7 steps
    B, T, H, D, Tmax = 4, 64, 8, 128, 64
    k, v = inputs.kv_tensor(B, T, H, D, 0, "k"), inputs.kv_tensor(B, T, H, D, 0, "v")
    s_k = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(B, T, H, D, 1, "k")))
    s_v = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(B, T, H, D, 1, "v")))
    kq, vq = np.zeros((B, H, Tmax, D // 2), np.uint8), np.zeros((B, H, Tmax, D // 2), np.uint8)
    tie_k, tie_v = np.ones((B, T, H, D), np.float32), np.ones((B, T, H, D), np.float32)
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq, vq, np.zeros(B, np.int32), tie_k, tie_v) == 0
    for x, s, q, tie in ((k, s_k, kq, tie_k), (v, s_v, vq, tie_v)):
        got = orc.unpack_int4(q).astype(np.int64).transpose(0, 2, 1, 3)  # [B,T,H,D]
        xd = x.to(torch.float64).numpy()
        ref = _rne_codes_f64(xd, s[None, None, :, None])
        diff = got != ref
        assert np.all(tie[diff] < 1e-4) and np.all(np.abs(got - ref)[diff] == 1)
        assert diff.sum() <= 1e-3 * diff.size, diff.sum()  # bf16 inputs over a max/7 step land next to ties often
        r = xd / s[None, None, :, None].astype(np.float64)
        inside = (tie > 1e-4) & (r > -8.5) & (r < 7.5)
        assert np.all(np.abs(got - r)[inside] < 0.5)
        assert np.all(got[r >= 7.5] == 7) and np.all(got[r <= -8.5] == -8)  # beyond the range the code clamps


# ---------------------------------------------------------------- integer GEMM
def test_gemm_brute_force_tiny():
    M, N, K = 3, 5, 8
    x = rng.integers(-8, 8, (M, K)).astype(np.int8)
    w = rng.integers(-8, 8, (N, K)).astype(np.int8)
    acc = orc.gemm_i4(orc.pack_int4(x), orc.pack_int4(w))
    for t, n in itertools.product(range(M), range(N)):
        assert acc[t, n] == sum(int(x[t, k]) * int(w[n, k]) for k in range(K))


def test_gemm_matches_int64_library_matmul_and_special_cases():
    M, N, K = 17, 23, 160
    x = rng.integers(-8, 8, (M, K)).astype(np.int8)
    w = rng.integers(-8, 8, (N, K)).astype(np.int8)
    acc = orc.gemm_i4(orc.pack_int4(x), orc.pack_int4(w))
    assert np.array_equal(acc, x.astype(np.int64) @ w.astype(np.int64).T)
    ones = np.ones((4, K), np.int8)
    assert np.all(orc.gemm_i4(orc.pack_int4(ones), orc.pack_int4(ones)) == K)
    lo = np.full((2, K), -8, np.int8)
    assert np.all(orc.gemm_i4(orc.pack_int4(lo), orc.pack_int4(lo)) == 64 * K)
    onehot = np.zeros((K, K), np.int8)
    onehot[np.arange(K), np.arange(K)] = 1
    assert np.array_equal(orc.gemm_i4(orc.pack_int4(onehot), orc.pack_int4(w)), w.T.astype(np.int32))


# ---------------------------------------------------------------- 8-bit activations (W4A8)
def test_quant_act8_hand_values_ties_clamp_and_scale():
    # no rotation, step 0.25: value / 0.25 decides the code by hand (Eq. 1 with N = 8, ties to even)
    vals = np.array([0.0, 0.125, 0.375, 0.625, -0.125, -0.375, 1.0, 31.75, 31.875, 40.0, -32.0, -32.125, -50.0, 0.3, -0.3, 7.8125])
    want = np.array([0, 0, 2, 2, 0, -2, 4, 127, 127, 127, -128, -128, -128, 1, -1, 31])
    x = np.tile(vals, (2, 8))  # K = 128
    got = orc.quant_act8(bf16_bits(x), 0, 0.25)
    assert got.dtype == np.int8 and np.array_equal(got, np.tile(want, (2, 8)))
    # idempotent on its own grid, monotone, full range reached
    grid = np.arange(-128, 128, dtype=np.float64)[None, :] * 0.25
    assert np.array_equal(orc.quant_act8(bf16_bits(grid), 0, 0.25)[0], np.arange(-128, 128))
    v = np.sort(rng.uniform(-40, 40, (1, 256)), axis=1)
    c = orc.quant_act8(bf16_bits(v), 0, 0.25).astype(int)
    assert np.all(np.diff(c) >= 0) and c.min() == -128 and c.max() == 127
    # the static step is max / 127 of the rotated rows at and after row_begin
    M, K, P = 6, 128, 2
    xb = inputs.bits(inputs.activations(M, K, seed=3, n_prefix=P))
    y = orc.rotate_bf16(xb, K)
    s = orc.calib_act_scale8(xb, K, row_begin=P)
    assert s == np.float32(np.abs(y[P:].astype(np.float32)).max() / 127.0)
    assert orc.calib_act_scale8(bf16_bits(np.zeros((2, K))), K) == 1.0
    # rotated case: within half a step of y / s, the largest element takes +-127, rows below row_begin stay zero
    q, tie = orc.quant_act8(xb, K, s, row_begin=P, want_tie_dist=True)
    r = y / np.float64(s)
    assert np.all(q[:P] == 0) and np.all(np.abs(q[P:] - r[P:]) <= 0.5 + 1e-9) and np.abs(q).max() == 127
    assert np.allclose(tie[P:], np.abs(r[P:] - np.floor(r[P:]) - 0.5), atol=1e-6)
    # eight more bits of resolution than the 4-bit code of the same tensor: the 4-bit code is the 8-bit one regrouped
    s4 = orc.calib_act_scale(xb, K, row_begin=P)
    assert np.isclose(float(s4) / float(s), 127.0 / 7.0, rtol=1e-6)


def test_gemm_i8i4_brute_force_and_library_matmul():
    M, N, K = 3, 5, 8
    x = rng.integers(-128, 128, (M, K)).astype(np.int8)
    w = rng.integers(-8, 8, (N, K)).astype(np.int8)
    acc = orc.gemm_i8i4(x, orc.pack_int4(w))
    for t, n in itertools.product(range(M), range(N)):
        assert acc[t, n] == sum(int(x[t, k]) * int(w[n, k]) for k in range(K))
    M, N, K = 9, 21, 192
    x = rng.integers(-128, 128, (M, K)).astype(np.int8)
    w = rng.integers(-8, 8, (N, K)).astype(np.int8)
    # nibbles unpacked here with numpy, not with the oracle's own routine
    pk = orc.pack_int4(w)
    lo, hi = (pk & 0xF).astype(np.int64), (pk >> 4).astype(np.int64)
    w_np = np.stack([np.where(lo > 7, lo - 16, lo), np.where(hi > 7, hi - 16, hi)], -1).reshape(N, K)
    assert np.array_equal(w_np, w)
    assert np.array_equal(orc.gemm_i8i4(x, pk), x.astype(np.int64) @ w_np.T)
    # a transposed or swapped operand shows up: one-hot rows pick weight columns, extremes hit the bound
    onehot = np.zeros((K, K), np.int8)
    onehot[np.arange(K), np.arange(K)] = 1
    assert np.array_equal(orc.gemm_i8i4(onehot, pk), w.T.astype(np.int32))
    lo8, lo4 = np.full((2, K), -128, np.int8), np.full((3, K), -8, np.int8)
    assert np.all(orc.gemm_i8i4(lo8, orc.pack_int4(lo4)) == 1024 * K)
    # 4-bit activations are a special case: the same codes as bytes give the W4A4 accumulator
    x4 = rng.integers(-8, 8, (M, K)).astype(np.int8)
    assert np.array_equal(orc.gemm_i8i4(x4, pk), orc.gemm_i4(orc.pack_int4(x4), pk))


# ---------------------------------------------------------------- per-token dynamic activations (O1)
def test_dynamic_per_token_quantizer_reduces_to_the_static_one_row_by_row():
    M, K, P = 7, 256, 2
    x = inputs.activations(M, K, seed=4, n_prefix=P)
    x[4] = 0
    xb = inputs.bits(x)
    s = orc.dyn_act_scale(xb, K, 1.0, row_begin=P)
    assert np.all(s[:P] == 0) and s[4] == 1.0
    codes, tie = orc.quant_act_rows(xb, K, np.where(s == 0, 1, s).astype(np.float32), row_begin=P, want_tie_dist=True)
    for m in range(P, M):
        # a single row is a one-row tensor: the per-tensor routines (pinned above) give its step and its codes
        assert s[m] == orc.calib_act_scale(xb[m:m + 1], K)
        ref, t1 = orc.quant_act(xb[m:m + 1], K, s[m], want_tie_dist=True)
        assert np.array_equal(codes[m:m + 1], ref) and np.array_equal(tie[m:m + 1], t1)
        if m != 4:
            assert np.abs(orc.unpack_int4(codes[m:m + 1])).max() == 7, "every token uses its full range"
    assert np.all(codes[:P] == 0) and np.all(codes[4] == 0)
    # the clipping factor is shared by the tokens of a layer and scales every step
    s_half = orc.dyn_act_scale(xb, K, 0.5, row_begin=P)
    live = np.arange(M) != 4
    assert np.allclose(s_half[P:][live[P:]], 0.5 * s[P:][live[P:]], rtol=2e-7)
    # dynamic means scale-free: a token multiplied by 2^k keeps its codes, its step takes the factor
    x2 = x.clone()
    x2[3] *= 8
    s2 = orc.dyn_act_scale(inputs.bits(x2), K, 1.0, row_begin=P)
    c2 = orc.quant_act_rows(inputs.bits(x2), K, np.where(s2 == 0, 1, s2).astype(np.float32), row_begin=P)
    assert s2[3] == 8 * s[3] and np.array_equal(c2, codes)
    # epilogue: a constant per-token step is the static epilogue
    acc = rng.integers(-(1 << 20), 1 << 20, (M, 9)).astype(np.int32)
    s_w = (rng.random(9) * 0.01 + 0.001).astype(np.float32)
    assert np.array_equal(orc.dequant_bf16_rows(acc, np.full(M, 0.37, np.float32), s_w), orc.dequant_bf16(acc, np.float32(0.37), s_w))
    got = orc.bf16_to_f64(orc.dequant_bf16_rows(acc, s.clip(1e-3), s_w))
    want = acc.astype(np.float64) * s.clip(1e-3).astype(np.float64)[:, None] * s_w.astype(np.float64)[None, :]
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-8 + 1e-30)


# ---------------------------------------------------------------- outlier tokens (Sec. 4.1, Eq. 2)
def test_outlier_tokens_hand_example_library_median_and_invariances():
    # six tokens with maxima 1, 2, 3, 4, 200, 0.25: median 2.5; R = 0.4, 0.8, 1.2, 1.6, 80, 0.1
    rows = np.zeros((6, 8))
    for i, m in enumerate([1, 2, 3, 4, 200, 0.25]):
        rows[i, i] = -m if i % 2 else m  # the maximum is of absolute values
        rows[i, 7] = 0.125 * (1 if i % 2 else -1)
    M, R, flags, med = orc.outlier_tokens(bf16_bits(rows))
    assert M.tolist() == [1, 2, 3, 4, 200, 0.25] and med == 2.5
    assert np.allclose(R, [0.4, 0.8, 1.2, 1.6, 80, 0.1], rtol=1e-6)
    assert flags.tolist() == [0, 0, 0, 0, 1, 2]  # 80 > 64 is an upper outlier, 1 / 0.1 = 10 > 8 a lower one
    # thresholds are strict and can be moved
    assert orc.outlier_tokens(bf16_bits(rows), eta1=80.0, eta2=10.0)[2].tolist() == [0, 0, 0, 0, 0, 0]
    assert orc.outlier_tokens(bf16_bits(rows), eta1=1.5, eta2=2.4)[2].tolist() == [2, 0, 0, 1, 1, 2]
    # against numpy on a random batch: odd and even token counts
    for T in (33, 64):
        x = inputs.activations(T, 256, seed=6)
        xb = inputs.bits(x)
        M, R, flags, med = orc.outlier_tokens(xb)
        Mref = np.abs(x.to(torch.float64).numpy()).max(1)
        assert np.array_equal(M, Mref.astype(np.float32)) and med == np.float32(np.median(Mref))
        assert np.allclose(R, Mref / np.median(Mref), rtol=2e-7)
        # token order does not matter, a common factor does not matter
        perm = rng.permutation(T)
        M2, R2, f2, med2 = orc.outlier_tokens(xb[perm])
        assert np.array_equal(R2, R[perm]) and np.array_equal(f2, flags[perm]) and med2 == med
        _, R3, f3, med3 = orc.outlier_tokens(inputs.bits(x * 4))
        assert np.array_equal(R3, R) and np.array_equal(f3, flags) and med3 == 4 * med
    # the synthetic prefix rows (1000 times larger) are exactly the upper outliers; a silent token is a lower one
    x = inputs.activations(40, 512, seed=1, n_prefix=4)
    x[17] *= 0.01
    flags = orc.outlier_tokens(inputs.bits(x))[2]
    assert flags[:4].tolist() == [1, 1, 1, 1] and flags[17] == 2 and int((flags != 0).sum()) == 5


# ---------------------------------------------------------------- Eq. 1 as printed: asymmetric with a zero point
def test_asymmetric_quantizer_hand_values_and_reduction_to_the_symmetric_one():
    # range [-1, 2.75]: s = 3.75 / 15 = 0.25, z = -round(-1 / 0.25) = 4
    s, z = orc.asym_params(-1.0, 2.75)
    assert s == 0.25 and z == 4
    # Eq. 1 prints the zero point with a floor: range [-1.0625, 2.6875] has s = 0.25, min / s = -4.25,
    # z = -floor(-4.25) = 5 (rounding would give 4); [-1.1875, 2.5625]: min / s = -4.75, z = 5 either way
    assert orc.asym_params(-1.0625, 2.6875) == (0.25, 5)
    assert orc.asym_params(-1.1875, 2.5625) == (0.25, 5)
    assert orc.asym_params(0.0625, 3.8125) == (0.25, 0)                # floor(0.25) = 0; a positive range keeps z = 0
    assert orc.asym_params(3.0, 3.0) == (1.0, 0)                       # a constant tensor
    assert orc.asym_params(0.0, 15.0) == (1.0, 0) and orc.asym_params(-15.0, 0.0) == (1.0, 15)
    vals = np.array([-1.0, 2.75, 0.125, 0.375, -0.125, -0.375, 5.0, -3.0, 0.0, 1.0, 0.3, -0.3])
    want = np.array([0, 15, 4, 6, 4, 2, 15, 0, 4, 8, 5, 3])           # round(x / s) + z, ties to even, clamp to [0, 15]
    pad = np.zeros(128 - len(vals))
    u = orc.quant_act_asym(bf16_bits(np.concatenate([vals, pad])[None, :]), 0, s, z)
    assert u.dtype == np.uint8 and u[0, :len(vals)].tolist() == want.tolist() and np.all(u[0, len(vals):] == 4)
    # dequantization s (u - z) is within half a step inside the range
    deq = s * (u[0, :len(vals)].astype(np.float64) - z)
    inside = (vals >= -1.0) & (vals <= 2.75)
    xb = orc.bf16_to_f64(bf16_bits(vals))
    assert np.all(np.abs(deq[inside] - xb[inside]) <= 0.125 + 1e-12)
    # with z = 8 the unsigned code is the signed code of the symmetric quantizer (pinned above) plus 8
    M, K = 5, 256
    xr = inputs.bits(inputs.activations(M, K, seed=7))
    s_sym = orc.calib_act_scale(xr, K)
    u8, tie = orc.quant_act_asym(xr, K, s_sym, 8, want_tie_dist=True)
    c_sym, tie_sym = orc.quant_act(xr, K, s_sym, want_tie_dist=True)
    assert np.array_equal(u8.astype(int) - 8, orc.unpack_int4(c_sym)) and np.array_equal(tie, tie_sym)
    # range of a rotated batch: prefix rows excluded; the codes of the calibration batch itself use the full range
    x = inputs.activations(12, K, seed=1, n_prefix=4)
    xb = inputs.bits(x)
    mn, mx = orc.calib_act_minmax(xb, K, row_begin=4)
    y = orc.rotate_bf16(xb, K)[4:].astype(np.float32)
    assert mn == y.min() and mx == y.max()
    s2, z2 = orc.asym_params(mn, mx)
    u2 = orc.quant_act_asym(xb, K, s2, z2, row_begin=4)
    # with the printed floor the zero point is ceil(-min / s): the minimum lands on code 0 or 1, and when it lands
    # on 1 the top of the range is clamped at 15 (one step lost there), never the bottom
    assert u2[4:].min() in (0, 1) and u2[4:].max() == 15 and np.all(u2[:4] == 0)
    assert z2 == int(np.ceil(-np.float64(mn) / np.float64(s2)))
    err = np.abs(s2 * (u2[4:].astype(np.float64) - z2) - y)
    top = u2[4:] == 15
    assert np.all(err[~top] <= 0.5 * s2 * (1 + 1e-5) + 1e-6) and np.all(err[top] <= 1.5 * s2 * (1 + 1e-5) + 1e-6)


def test_grid_search_for_s_and_z_brute_force_and_never_worse_than_max_min():
    # candidates: the first one is the max-min pair (pinned above), the factors step down to lo
    mn, mx = np.float32(-1.0), np.float32(2.75)
    cs, cz = orc.grid_candidates(mn, mx, 3, 0.5)
    assert (cs[0], cz[0]) == orc.asym_params(mn, mx)
    # gamma, beta in {1, 0.75, 0.5}: s = (gamma * 2.75 + beta) / 15, z = -floor(-beta / s), by hand for two of them
    assert cs[4] == np.float32((np.float32(0.75 * 2.75) + np.float32(0.75)) / np.float32(15))        # i = j = 1
    assert cz[4] == int(-np.floor(np.float32(-0.75) / cs[4])) and cs[8] == np.float32(0.5) * cs[0] and cz[8] == cz[0]
    assert orc.grid_candidates(np.float32(0.0), np.float32(0.0), 2, 0.5)[0].tolist() == [1.0] * 4    # empty range
    # the squared error against an independent numpy evaluation on a tiny tensor without rotation
    x = rng.standard_normal((3, 128)) * 2.0 + 0.7
    x[1, 5] = 40.0                                   # one far value: clipping it pays
    xb = bf16_bits(x)
    y = orc.bf16_to_f64(xb)
    lo_, hi_ = np.float32(y.min()), np.float32(y.max())
    n, lo = 6, 0.1
    s_best, z_best, sse = orc.grid_search_act(xb, 0, n, lo)
    cs, cz = orc.grid_candidates(lo_, hi_, n, lo)
    ref = np.empty(n * n)
    for c in range(n * n):
        sd = np.float64(cs[c])
        u = np.clip(np.rint(y / sd) + cz[c], 0, 15)
        ref[c] = ((y - sd * (u - cz[c])) ** 2).sum()
        assert orc.quant_sse_asym(xb, 0, cs[c], cz[c]) == pytest.approx(ref[c], rel=1e-12)
    assert np.allclose(sse, ref, rtol=1e-12) and (s_best, z_best) == (cs[ref.argmin()], int(cz[ref.argmin()]))
    assert ref.min() <= ref[0] and ref.argmin() != 0, "with an outlier in the tensor the max-min pair is not the best one"
    # a tensor that lies on a candidate's grid is reproduced without error by that candidate
    s0, z0 = np.float32(0.25), 5
    grid_vals = (np.arange(16) - z0) * 0.25
    xg = bf16_bits(np.tile(grid_vals, (2, 8)))
    assert orc.quant_sse_asym(xg, 0, s0, z0) == 0.0
    sg, zg, sse_g = orc.grid_search_act(xg, 0, 4, 0.5)
    assert sse_g[0] == 0.0 and (sg, zg) == (s0, z0), "max-min already is exact here and comes first"
    # rotation and prefix rows: the error is taken over the rotated rows at and after row_begin only
    xr = inputs.bits(inputs.activations(10, 256, seed=1, n_prefix=4))
    yr = orc.rotate_bf16(xr, 256)[4:]
    s1, z1 = orc.asym_params(np.float32(yr.astype(np.float32).min()), np.float32(yr.astype(np.float32).max()))
    u = np.clip(np.rint(yr / np.float64(s1)) + z1, 0, 15)
    assert orc.quant_sse_asym(xr, 256, s1, z1, row_begin=4) == pytest.approx(((yr - np.float64(s1) * (u - z1)) ** 2).sum(), rel=1e-12)


def test_grid_search_for_the_dynamic_clipping_factor_brute_force():
    # Sec. 3: for per-token dynamic quantization one clipping factor is shared by all tokens and chosen by squared error.
    # Independent evaluation in numpy on a small tensor: no rotation first, then with an explicit Hadamard matrix.
    n, lo = 9, 0.2
    x = rng.standard_normal((6, 128))
    x[:, 3] *= 12.0                                   # a heavy column: every row's maximum is far from its bulk
    xb = bf16_bits(x)
    y = orc.bf16_to_f64(xb)
    g, cand, sse = orc.grid_search_clip_dyn(xb, 0, n, lo)
    step = np.float32(np.float32(1.0 - np.float32(lo)) / np.float32(n - 1))
    assert cand.tolist() == [float(np.float32(1.0) - np.float32(np.float32(i) * step)) for i in range(n)] and cand[0] == 1.0
    ref = np.empty(n)
    for i in range(n):
        s = (np.float64(cand[i]) * np.abs(y.astype(np.float32).astype(np.float64)).max(axis=1) / 7.0).astype(np.float32).astype(np.float64)
        q = np.clip(np.rint(y / s[:, None]), -8, 7)
        ref[i] = ((y - s[:, None] * q) ** 2).sum()
    assert np.allclose(sse, ref, rtol=1e-12) and g == cand[ref.argmin()]
    assert ref.argmin() != 0, "with a heavy tail clipping pays: the unclipped step is not the best one"
    # candidate 0 is the unclipped quantizer that orc_dyn_act_scale / orc_quant_act_rows define
    s1 = orc.dyn_act_scale(xb, 0)
    codes = orc.unpack_int4(orc.quant_act_rows(xb, 0, s1)).astype(np.float64)
    assert sse[0] == pytest.approx(((y - s1.astype(np.float64)[:, None] * codes) ** 2).sum(), rel=1e-12)
    # values already on the unclipped grid: no error at gamma = 1, which then wins as the first of the equals or alone
    xg = bf16_bits(np.tile(np.arange(-7, 8, dtype=np.float64) * 0.5, (2, 8))[:, :64].repeat(2, axis=1))
    gg, _, sse_g = orc.grid_search_clip_dyn(xg, 0, 4, 0.5)
    assert sse_g[0] == 0.0 and gg == 1.0
    # rotation and prefix rows: rotated rows at and after row_begin, against the explicit Sylvester matrix
    H = np.array([[1.0]])
    while H.shape[0] < 64:
        H = np.block([[H, H], [H, -H]])
    xr = inputs.bits(inputs.activations(9, 128, seed=3, n_prefix=4))
    yr = (orc.bf16_to_f64(xr).reshape(9, 2, 64) @ H / 8.0).reshape(9, 128)[4:]
    _, cand_r, sse_r = orc.grid_search_clip_dyn(xr, 64, 5, 0.5, row_begin=4)
    for i in (0, 2, 4):
        s = (np.float64(cand_r[i]) * np.abs(yr.astype(np.float32).astype(np.float64)).max(axis=1) / 7.0).astype(np.float32).astype(np.float64)
        q = np.clip(np.rint(yr / s[:, None]), -8, 7)
        assert sse_r[i] == pytest.approx(((yr - s[:, None] * q) ** 2).sum(), rel=1e-9)


def test_gemm_asym_is_the_dequantized_product():
    M, N, K, z = 7, 11, 96, 5
    u = rng.integers(0, 16, (M, K)).astype(np.uint8)
    w = rng.integers(-8, 8, (N, K)).astype(np.int8)
    acc = orc.gemm_asym(u, z, orc.pack_int4(w))
    assert np.array_equal(acc, (u.astype(np.int64) - z) @ w.astype(np.int64).T)
    for t, n in itertools.product(range(2), range(3)):
        assert acc[t, n] == sum((int(u[t, k]) - z) * int(w[n, k]) for k in range(K))
    # zero point 8: the symmetric GEMM on the codes u - 8
    assert np.array_equal(orc.gemm_asym(u, 8, orc.pack_int4(w)), orc.gemm_i4(orc.pack_int4((u.astype(int) - 8).astype(np.int8)), orc.pack_int4(w)))
    # the correction-term identity the GPU epilogue uses: sum (u - z) w = sum (u - 8) w - (z - 8) sum_k w
    raw = orc.gemm_i4(orc.pack_int4((u.astype(int) - 8).astype(np.int8)), orc.pack_int4(w))
    assert np.array_equal(acc, raw - (z - 8) * w.astype(np.int64).sum(1)[None, :])


def test_dequant_epilogue_closed_form_and_one_rounding():
    acc = np.array([[3, -5, 0, 1 << 20]], np.int32)
    s_w = np.array([0.25, 0.5, 7.0, 2.0**-10], np.float32)
    out = orc.bf16_to_f64(orc.dequant_bf16(acc, 0.5, s_w))
    assert out.tolist() == [[0.375, -1.25, 0.0, 512.0]]
    acc = rng.integers(-200000, 200000, (8, 16)).astype(np.int32)
    s_w = (rng.random(16) * 0.01 + 1e-3).astype(np.float32)
    s_a = np.float32(0.0371)
    got = orc.bf16_to_f64(orc.dequant_bf16(acc, s_a, s_w))
    exact = acc.astype(np.float64) * np.float64(s_a) * s_w.astype(np.float64)[None, :]
    assert np.all(np.abs(got - exact) <= np.abs(exact) * 2.0**-8 + 1e-300)  # half a bf16 ulp (8 significant bits)


# ---------------------------------------------------------------- KV cache
def test_kv_scale_and_append():
    B, T, H, D, Tmax = 2, 3, 2, 16, 8
    k = inputs.kv_tensor(B, T, H, D, 0, "k")
    v = inputs.kv_tensor(B, T, H, D, 0, "v")
    kc = inputs.kv_tensor(4, 8, H, D, 1, "k")
    s_k = orc.calib_kv_scale(inputs.bits(kc))
    kcf = kc.to(torch.float64).numpy()
    assert np.array_equal(s_k, (np.abs(kcf).max(axis=(0, 1, 3)) / 7).astype(np.float32))
    s_v = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(4, 8, H, D, 1, "v")))
    kq = np.full((B, H, Tmax, D // 2), 0xEE, np.uint8)
    vq = np.full((B, H, Tmax, D // 2), 0xEE, np.uint8)
    length = np.array([1, 4], np.int32)
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq, vq, length) == 0
    assert length.tolist() == [4, 7]
    kcodes = orc.unpack_int4(kq)
    kf = k.to(torch.float64).numpy()
    for b, l0 in enumerate([1, 4]):
        for h in range(H):
            r = kf[b, :, h, :] / np.float64(s_k[h])
            got = kcodes[b, h, l0:l0 + T]
            assert np.all(np.abs(got - np.clip(r, -8, 7)) <= 0.5 + 1e-6)  # decided in fp32
            assert np.all(kq[b, h, :l0] == 0xEE) and np.all(kq[b, h, l0 + T:] == 0xEE)  # nothing else touched
    # a sequence that would overflow Tmax is refused and nothing moves
    before = kq.copy()
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq, vq, length) == 1
    assert np.array_equal(kq, before) and length.tolist() == [4, 7]


# ---------------------------------------------------------------- attention (Eq. 3)
def _attn_setup(B=2, Hq=4, Hkv=2, D=16, P=2, T=9, Tmax=12, mag=1.0, seed=0):
    q = inputs.queries(B, Hq, D, seed)
    pk = inputs.prefix_kv(Hkv, P, D, seed, "k", mag)
    pv = inputs.prefix_kv(Hkv, P, D, seed, "v", mag)
    kq = rng.integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    vq = rng.integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    s_k = (rng.random(Hkv) * 0.3 + 0.1).astype(np.float32)
    s_v = (rng.random(Hkv) * 0.3 + 0.1).astype(np.float32)
    length = np.array([T, T - 4][:B], np.int32)
    return q, pk, pv, kq, vq, s_k, s_v, length


def _library_attention(q, pk, pv, kq, vq, s_k, s_v, length, sm):
    """Textbook softmax attention with torch on the dequantized tensors (float64)."""
    B, Hq, D = q.shape
    Hkv = pk.shape[0]
    out = np.zeros((B, Hq, D))
    kd = orc.unpack_int4(kq).astype(np.float64) * s_k.astype(np.float64)[None, :, None, None]
    vd = orc.unpack_int4(vq).astype(np.float64) * s_v.astype(np.float64)[None, :, None, None]
    for b in range(B):
        for g in range(Hq):
            h = g // (Hq // Hkv)
            K = torch.cat([pk[h].double(), torch.from_numpy(kd[b, h, :length[b]])])
            V = torch.cat([pv[h].double(), torch.from_numpy(vd[b, h, :length[b]])])
            p = torch.softmax(K @ q[b, g].double() * sm, dim=0)
            out[b, g] = (p @ V).numpy()
    return out


def test_decode_attention_equals_library_softmax_attention():
    q, pk, pv, kq, vq, s_k, s_v, length = _attn_setup()
    sm = 1 / math.sqrt(16)
    out, out64 = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq, vq, s_k, s_v, length, sm, want_f64=True)
    ref = _library_attention(q, pk, pv, kq, vq, s_k, s_v, length, sm)
    assert np.allclose(out64, ref, rtol=1e-12, atol=1e-13)
    assert np.array_equal(out, orc.f64_to_bf16(out64))
    # no prefix at all: plain attention over the dequantized cache
    pk0, pv0 = pk[:, :0], pv[:, :0]
    _, o0 = orc.decode_attn(inputs.bits(q), inputs.bits(pk0), inputs.bits(pv0), kq, vq, s_k, s_v, length, sm, want_f64=True)
    assert np.allclose(o0, _library_attention(q, pk0, pv0, kq, vq, s_k, s_v, length, sm), rtol=1e-12, atol=1e-13)
    # empty cache: attention over the full-precision prefix only
    _, o1 = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq, vq, s_k, s_v, np.zeros(2, np.int32), sm, want_f64=True)
    assert np.allclose(o1, _library_attention(q, pk, pv, kq, vq, s_k, s_v, [0, 0], sm), rtol=1e-12, atol=1e-13)


def test_decode_attention_closed_forms():
    B, Hq, Hkv, D, P, T, Tmax = 1, 4, 2, 16, 0, 6, 6
    q = inputs.queries(B, Hq, D, 3)
    pk = torch.zeros((Hkv, 0, D), dtype=torch.float16)
    vq = rng.integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    s = np.array([0.5, 0.25], np.float32)
    length = np.array([T], np.int32)
    # all-zero keys -> uniform probabilities -> output is the mean of V
    kq = np.zeros((B, Hkv, Tmax, D // 2), np.uint8)
    _, o = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pk), kq, vq, s, s, length, 0.25, want_f64=True)
    vd = orc.unpack_int4(vq).astype(np.float64) * s.astype(np.float64)[None, :, None, None]
    for g in range(Hq):
        assert np.allclose(o[0, g], vd[0, g // 2].mean(0), rtol=1e-13)
    # one dominant key -> output is that key's value row; equal queries in a GQA group -> equal outputs
    qd = torch.zeros((1, Hq, D), dtype=torch.bfloat16)
    qd[..., 0] = 100.0
    kc = np.zeros((B, Hkv, Tmax, D), np.int8)
    kc[:, :, 3, 0] = 7
    _, o = orc.decode_attn(inputs.bits(qd), inputs.bits(pk), inputs.bits(pk), orc.pack_int4(kc), vq, s, s, length, 1.0, want_f64=True)
    for g in range(Hq):
        assert np.allclose(o[0, g], vd[0, g // 2, 3], rtol=1e-9)
    assert np.array_equal(o[0, 0], o[0, 1]) and np.array_equal(o[0, 2], o[0, 3])


def test_decode_attention_key_permutation_invariance():
    q, pk, pv, kq, vq, s_k, s_v, length = _attn_setup(B=1, T=9)
    sm = 0.25
    _, o = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq, vq, s_k, s_v, length, sm, want_f64=True)
    perm = rng.permutation(int(length[0]))
    kq2, vq2 = kq.copy(), vq.copy()
    kq2[:, :, :length[0]] = kq[:, :, perm]
    vq2[:, :, :length[0]] = vq[:, :, perm]
    _, o2 = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq2, vq2, s_k, s_v, length, sm, want_f64=True)
    assert np.allclose(o, o2, rtol=1e-12, atol=1e-14)


def test_prefill_attention_is_causal_decode_per_row():
    T, Hq, Hkv, D, P, Tmax = 7, 4, 2, 16, 2, 8
    qt = inputs.normal(5, inputs.STREAM_Q, (T, Hq, D), dtype=torch.bfloat16)
    pk = inputs.prefix_kv(Hkv, P, D, 0, "k", 1.0)
    pv = inputs.prefix_kv(Hkv, P, D, 0, "v", 1.0)
    kq = rng.integers(0, 256, (Hkv, Tmax, D // 2)).astype(np.uint8)
    vq = rng.integers(0, 256, (Hkv, Tmax, D // 2)).astype(np.uint8)
    s_k = np.array([0.2, 0.3], np.float32)
    s_v = np.array([0.4, 0.1], np.float32)
    out, out64 = orc.prefill_attn(inputs.bits(qt), inputs.bits(pk), inputs.bits(pv), kq, vq, s_k, s_v, 0.25, want_f64=True)
    assert np.array_equal(out, orc.f64_to_bf16(out64))
    for t in range(T):
        ref, ref64 = orc.decode_attn(inputs.bits(qt[t:t + 1]), inputs.bits(pk), inputs.bits(pv), kq[None], vq[None], s_k, s_v,
                                     np.array([t + 1], np.int32), 0.25, want_f64=True)
        assert np.array_equal(out[t], ref[0]) and np.array_equal(out64[t], ref64[0])
    # without a prefix the first token attends to itself only: its output is its own value row
    out0 = orc.prefill_attn(inputs.bits(qt), inputs.bits(pk[:, :0]), inputs.bits(pv[:, :0]), kq, vq, s_k, s_v, 0.25)
    vd = orc.unpack_int4(vq).astype(np.float64) * s_v.astype(np.float64)[:, None, None]
    for g in range(Hq):
        assert np.array_equal(out0[0, g], orc.f64_to_bf16(vd[g // 2, 0]))


# ---------------------------------------------------------------- group-wise dynamic KV4 (Table 1, O1)
def test_groupwise_dynamic_kv_steps_codes_and_attention():
    B, T, H, D, Tmax, Hq, P = 2, 5, 2, 128, 8, 4, 2
    k, v = inputs.kv_tensor(B, T, H, D, 0, "k"), inputs.kv_tensor(B, T, H, D, 0, "v")
    k[1, 2, 0] = 0                                        # an all-zero vector: step 1, codes 0
    kq, vq = np.full((B, H, Tmax, D // 2), 0xEE, np.uint8), np.full((B, H, Tmax, D // 2), 0xEE, np.uint8)
    sk, sv = np.full((B, H, Tmax), -1, np.float32), np.full((B, H, Tmax), -1, np.float32)
    length = np.array([1, 3], np.int32)
    assert orc.kv4_append_dyn(inputs.bits(k), inputs.bits(v), kq, vq, sk, sv, length) == 0 and length.tolist() == [6, 8]
    kf, vf = k.to(torch.float32).numpy(), v.to(torch.float32).numpy()
    for b, l0 in enumerate([1, 3]):
        # one step per (token, head) vector = its own max / 7 (fp32); positions outside the append untouched
        mk = np.abs(kf[b]).max(-1).T                      # [H, T]
        assert np.array_equal(sk[b, :, l0:l0 + T], np.where(mk == 0, np.float32(1), mk / np.float32(7)).astype(np.float32))
        assert np.array_equal(sv[b, :, l0:l0 + T], (np.abs(vf[b]).max(-1).T / np.float32(7)).astype(np.float32))
        assert np.all(sk[b, :, :l0] == -1) and np.all(kq[b, :, :l0] == 0xEE) and np.all(sk[b, :, l0 + T:] == -1)
        codes = orc.unpack_int4(kq[b, :, l0:l0 + T]).astype(np.float64)           # [H, T, D]
        r = kf[b].transpose(1, 0, 2).astype(np.float64) / sk[b, :, l0:l0 + T, None].astype(np.float64)
        assert np.all(np.abs(codes - r) <= 0.5 + 1e-6)
        nz = mk > 0
        assert np.all(np.abs(codes).max(-1)[nz] == 7), "every vector uses its full range: that is what dynamic means"
    assert np.all(orc.unpack_int4(kq[1, 0, 3 + 2]) == 0) and sk[1, 0, 3 + 2] == 1.0
    assert orc.kv4_append_dyn(inputs.bits(k), inputs.bits(v), kq, vq, sk, sv, length) == 1                       # would pass Tmax
    # scale-free per vector: a vector multiplied by 2^p keeps its codes, its step takes the factor
    k2 = k.clone()
    k2[0, 1, 1] *= 8
    kq2, sk2 = np.zeros_like(kq), np.zeros_like(sk)
    orc.kv4_append_dyn(inputs.bits(k2), inputs.bits(v), kq2, np.zeros_like(vq), sk2, np.zeros_like(sv), np.array([1, 3], np.int32))
    assert np.array_equal(kq2[0, 1, 2], kq[0, 1, 2]) and sk2[0, 1, 2] == 8 * sk[0, 1, 2] and np.array_equal(kq2[1, :, 3:8], kq[1, :, 3:8])
    # with equal maxima in every vector the steps are all equal and the path is the static one, bit for bit
    ke = k.clone()
    ke[..., 0] = 9.0
    s_stat = np.full(H, np.float32(9.0) / np.float32(7), np.float32)
    kq_d, vq_d, sk_d, sv_d = np.zeros_like(kq), np.zeros_like(vq), np.zeros_like(sk), np.zeros_like(sv)
    orc.kv4_append_dyn(inputs.bits(ke), inputs.bits(ke), kq_d, vq_d, sk_d, sv_d, np.zeros(B, np.int32))
    kq_s, vq_s = np.zeros_like(kq), np.zeros_like(vq)
    orc.kv4_append(inputs.bits(ke), inputs.bits(ke), s_stat, s_stat, kq_s, vq_s, np.zeros(B, np.int32))
    assert np.array_equal(kq_d, kq_s) and np.array_equal(vq_d, vq_s) and np.all(sk_d[:, :, :T] == s_stat[0])
    q = inputs.queries(B, Hq, D, 0)
    pk, pv = inputs.prefix_kv(H, P, D, 0, "k", 1.0), inputs.prefix_kv(H, P, D, 0, "v", 1.0)
    lens = np.full(B, T, np.int32)
    o_d, o64_d = orc.decode_attn_dyn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_d, vq_d, sk_d, sv_d, lens, 0.1)
    o_s, o64_s = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_s, vq_s, s_stat, s_stat, lens, 0.1, want_f64=True)
    assert np.array_equal(o_d, o_s) and np.array_equal(o64_d, o64_s)
    # general steps: a library softmax attention over the tensors dequantized with their own per-key steps
    lens = np.array([6, 8], np.int32)
    _, o64 = orc.decode_attn_dyn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq, vq, sk, sv, lens, 0.1)
    kd = orc.unpack_int4(kq).astype(np.float64) * sk.astype(np.float64)[..., None]
    vd = orc.unpack_int4(vq).astype(np.float64) * sv.astype(np.float64)[..., None]
    for b in range(B):
        for g in range(Hq):
            h = g // (Hq // H)
            K = torch.cat([pk[h].double(), torch.from_numpy(kd[b, h, :lens[b]])])
            V = torch.cat([pv[h].double(), torch.from_numpy(vd[b, h, :lens[b]])])
            p = torch.softmax(K @ q[b, g].double() * 0.1, dim=0)
            assert np.allclose(o64[b, g], (p @ V).numpy(), rtol=1e-12, atol=1e-13)
    # prefill = the causal rows of the decode form
    qt = inputs.normal(5, inputs.STREAM_Q, (6, Hq, D), dtype=torch.bfloat16)
    op, op64 = orc.prefill_attn_dyn(inputs.bits(qt), inputs.bits(pk), inputs.bits(pv), kq[0], vq[0], sk[0], sv[0], 0.1)
    for t in range(6):
        od, od64 = orc.decode_attn_dyn(inputs.bits(qt[t:t + 1]), inputs.bits(pk), inputs.bits(pv), kq[:1], vq[:1], sk[:1], sv[:1],
                                       np.array([t + 1], np.int32), 0.1)
        assert np.array_equal(op[t], od[0]) and np.array_equal(op64[t], od64[0])


# ---------------------------------------------------------------- block glue
def test_rope_matches_complex_rotation_and_relative_property():
    T, H, D, theta = 6, 2, 16, 500000.0
    x = inputs.normal(9, inputs.STREAM_Q, (T, H, D), dtype=torch.bfloat16)
    y = orc.bf16_to_f64(orc.rope(inputs.bits(x), 4, theta))
    xd = x.to(torch.float64).numpy()
    z = xd[..., :D // 2] + 1j * xd[..., D // 2:]
    freq = theta ** (-np.arange(D // 2) * 2.0 / D)
    pos = (4 + np.arange(T))[:, None, None]
    zr = z * np.exp(1j * pos * freq[None, None, :])
    ref = np.concatenate([zr.real, zr.imag], -1)
    assert np.all(np.abs(y - ref) <= np.abs(ref) * 2.0**-8 + 1e-30)
    # position 0 is the identity
    y0 = orc.rope(inputs.bits(x[:1]), 0, theta)
    assert np.array_equal(y0, inputs.bits(x[:1]))
    # <rope(a, m), rope(b, n)> depends on m - n only (checked through the complex form, in double)
    a, b = z[0, 0], z[1, 0]
    d1 = np.real(np.sum(a * np.exp(1j * 7 * freq) * np.conj(b * np.exp(1j * 3 * freq))))
    d2 = np.real(np.sum(a * np.exp(1j * 14 * freq) * np.conj(b * np.exp(1j * 10 * freq))))
    assert abs(d1 - d2) < 1e-10


def test_rope_rotate_is_complex_rotation_times_library_hadamard():
    """R3 (App. B): after the rotary embedding every head is multiplied by H_D / sqrt(D)."""
    T, H, D, theta = 5, 3, 128, 500000.0
    x = inputs.normal(11, inputs.STREAM_Q, (T, H, D), dtype=torch.bfloat16)
    y = orc.bf16_to_f64(orc.rope_rotate(inputs.bits(x), 4, theta))
    xd = x.to(torch.float64).numpy()
    z = xd[..., :D // 2] + 1j * xd[..., D // 2:]
    freq = theta ** (-np.arange(D // 2) * 2.0 / D)
    zr = z * np.exp(1j * (4 + np.arange(T))[:, None, None] * freq[None, None, :])
    roped = np.concatenate([zr.real, zr.imag], -1)
    ref = roped @ hadamard(D).astype(np.float64) / math.sqrt(D)
    assert np.all(np.abs(y - ref) <= np.abs(ref) * 2.0**-8 + 1e-30), "one rounding to bf16 of the exact product"
    # at position 0 the rotary part is the identity: what is left is the plain rotation of the input
    y0 = orc.bf16_to_f64(orc.rope_rotate(inputs.bits(x[:1]), 0, theta))
    r0 = orc.rotate_bf16(inputs.bits(x[:1]).reshape(H, D), D)
    assert np.all(np.abs(y0.reshape(H, D) - r0) <= np.abs(r0) * 2.0**-8 + 1e-30)
    # computational invariance: scores between rotated q and k equal the scores without R3 (up to the bf16 store)
    plain = orc.bf16_to_f64(orc.rope(inputs.bits(x), 4, theta))
    s_rot = np.einsum("thd,shd->hts", y, y)
    s_plain = np.einsum("thd,shd->hts", plain, plain)
    assert np.allclose(s_rot, s_plain, rtol=0, atol=2.0**-7 * np.abs(s_plain).max())
    # a unit vector in dim j at position 0 becomes column j of H / sqrt(D): every entry +-1/sqrt(128), sign by popcount
    e = np.zeros((1, 1, D))
    e[0, 0, 5] = 1.0
    ye = orc.bf16_to_f64(orc.rope_rotate(bf16_bits(e), 0, theta))[0, 0]
    sign = np.array([(-1.0) ** bin(5 & j).count("1") for j in range(D)])
    assert np.array_equal(ye, orc.bf16_to_f64(bf16_bits(sign / math.sqrt(D))))


def test_rmsnorm_silu_add_closed_forms():
    x = inputs.activations(5, 64, seed=0)
    g = torch.ones(64, dtype=torch.bfloat16)
    y = orc.bf16_to_f64(orc.rmsnorm(inputs.bits(x), inputs.bits(g), 0.0))
    assert np.allclose(np.sqrt((y**2).mean(1)), 1.0, atol=4e-3)
    y2 = orc.bf16_to_f64(orc.rmsnorm(inputs.bits(x * 4), inputs.bits(g), 0.0))
    assert np.array_equal(y, y2)  # scale invariance (power-of-two scaling is exact in bf16)
    ref = torch.nn.functional.rms_norm(x.double(), (64,), eps=1e-5).numpy()
    got = orc.bf16_to_f64(orc.rmsnorm(inputs.bits(x), inputs.bits(g), 1e-5))
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0**-8)
    gate = torch.tensor([0.0, 30.0, -30.0, 1.0, -1.0], dtype=torch.bfloat16)
    up = torch.tensor([5.0, 2.0, 2.0, 3.0, 3.0], dtype=torch.bfloat16)
    s = orc.bf16_to_f64(orc.silu_mul(inputs.bits(gate), inputs.bits(up)))
    ref = (torch.nn.functional.silu(gate.double()) * up.double()).numpy()
    assert s[0] == 0.0 and s[1] == 60.0 and abs(s[2]) < 1e-11
    assert np.all(np.abs(s - ref) <= np.abs(ref) * 2.0**-8 + 1e-30)
    a = torch.tensor([1.0, 2.5, -3.0], dtype=torch.bfloat16)
    b = torch.tensor([0.5, 0.25, 3.0], dtype=torch.bfloat16)
    assert orc.bf16_to_f64(orc.add(inputs.bits(a), inputs.bits(b))).tolist() == [1.5, 2.75, 0.0]


# ---------------------------------------------------------------- input generator sanity (no method arithmetic there)
def test_input_generator_is_deterministic_and_sliceable():
    a = inputs.normal(3, inputs.STREAM_ACT, (1000,))
    b = inputs.normal(3, inputs.STREAM_ACT, (1000,))
    assert torch.equal(a, b)
    c = inputs.normal(3, inputs.STREAM_ACT, (400,), offset=600)
    assert torch.equal(a[600:], c)
    big = inputs.normal(4, inputs.STREAM_ACT, (200000,))
    assert abs(float(big.mean())) < 0.01 and abs(float(big.std()) - 1.0) < 0.01
    assert not torch.equal(inputs.normal(3, inputs.STREAM_ACT, (10,)), inputs.normal(3, inputs.STREAM_K, (10,)))
